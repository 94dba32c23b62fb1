"""The library's environment switches select alternative code paths (debugging and tuning aids).  Each of them is
run once here, in a process of its own with the variable set, through parity tests of the tiny pair: a path that is
kept must stay correct."""
import os
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu

torch = pytest.importorskip("torch")

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
# what the switch changes -> the tests that exercise it
SINGLE = "test_tiny_models_teacher_forced and 64 or test_hand_traced_stream_on_device"
BATCH = "test_batched_decode_tiny or test_batched_generation_in_rounds"
CASES = [
    ("ST_HOST_LOOP", "1", "test_hand_traced_stream_on_device or test_tiny_pair_fully_forced_routing_and_logits"),
    ("ST_MULTI_KERNEL", "1", SINGLE),
    ("ST_SIMT_GEMM", "1", SINGLE),
    ("ST_SIMT_ATTN", "1", SINGLE),
    ("ST_PDL", "0", SINGLE + " or " + BATCH),
    ("ST_AB_TILE", "128", BATCH),
    ("ST_BATCH_SEQUENTIAL", "1", "test_three_takeovers_on_device or test_every_delimiter_variant_on_device"),
    ("ST_BATCH_GRAPH", "0", BATCH),
    ("ST_BATCH_OVERLAP", "0", "test_batched_generation_in_rounds"),
    ("ST_MEGA_STAGES", "2", SINGLE),
    ("ST_DOWN_SLAB", "1", SINGLE),
    ("ST_MEGA_UNIT_KEYS", "32", "test_decode_from_empty_cache_and_long_context"),
]


@pytest.mark.parametrize("var,value,select", CASES, ids=[c[0] for c in CASES])
def test_switch(var, value, select):
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    env = dict(os.environ, **{var: value})
    r = subprocess.run([sys.executable, "-m", "pytest", os.path.join(ROOT, "tests", "test_gpu_parity.py"), "-x", "-q", "-m", "gpu",
                        "-k", select, "-p", "no:cacheprovider"], env=env, cwd=ROOT, capture_output=True, text=True, timeout=600)
    tail = (r.stdout + r.stderr)[-1500:]
    assert r.returncode == 0, f"{var}={value}: {tail}"
    assert " passed" in r.stdout and "no tests ran" not in r.stdout, tail


def test_time_gemv_runs_every_projection():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    import ctypes as C
    from paper_2504_12329_b200 import binding as B, workloads as W
    m = B.Model(W.TINY_L.as_dict(), seed=0, tag=1, max_tokens=128)
    for which in range(5):
        sec = C.c_double(0.0)
        assert B.lib().st_time_gemv(m.h, which, 4, C.byref(sec)) == 0
        assert 0.0 < sec.value < 1e-2
    bad = C.c_double(0.0)
    assert B.lib().st_time_gemv(m.h, 7, 4, C.byref(bad)) == B.ST_ERR_ARG
    assert m.st_last_device_status() == 0
    m.close()
