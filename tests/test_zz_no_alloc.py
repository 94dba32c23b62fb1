"""The allocation-free sampling entry point against the regular decode step (collected last).

st_argmax_static serves callers that cannot allocate device memory -- for instance code that runs
while another component holds the whole memory pool, or inside a region where an allocation would
synchronise the device.  Its scratch is an array built into the library, shared by every call, so
the check runs it twice in a row: the second call must not be disturbed by what the first left.
"""
import numpy as np
import pytest

from paper_2504_12329_b200 import workloads as W

pytestmark = pytest.mark.gpu

torch = pytest.importorskip("torch")


def test_static_argmax_matches_decode_step_twice():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2504_12329_b200 import binding as B, build
    build.build()   # no-op when the in-tree library is newer than its sources
    shape = W.TINY_L.as_dict()
    m = B.Model(shape, seed=0, tag=1, max_tokens=128)
    slot = m.st_seq_alloc()
    m.st_prefill(slot, W.prompt_ids(3, 9, shape["vocab"]))
    logits = torch.empty(shape["vocab"], dtype=torch.float32, device="cuda")
    want = torch.empty(1, dtype=torch.int32, device="cuda")
    got = torch.full((1,), -1, dtype=torch.int32, device="cuda")
    tok = torch.empty(1, dtype=torch.int32, device="cuda")
    stream = torch.cuda.current_stream().cuda_stream
    for step, t in enumerate((17, 501)):              # two calls in a row, different logits
        tok.fill_(t)
        m.st_decode_step([slot], tok, logits, want)   # existing entry point: logits and its argmax
        B.st_argmax_static(logits, shape["vocab"], got, stream)
        torch.cuda.synchronize()
        assert int(got.item()) == int(want.item()), f"call {step}"
        assert int(got.item()) == int(np.argmax(logits.cpu().numpy()))
        # a prefix of the vector: ids beyond n never win
        B.st_argmax_static(logits, 100, got, stream)
        torch.cuda.synchronize()
        assert int(got.item()) == int(np.argmax(logits.cpu().numpy()[:100]))
    # ties go to the lowest id, as in the decode step
    flat = torch.zeros(4096, dtype=torch.float32, device="cuda")
    flat[1234] = 1.0
    flat[77] = 1.0
    B.st_argmax_static(flat, 4096, got, stream)
    torch.cuda.synchronize()
    assert int(got.item()) == 77
    # sizes that leave some of the 64 CTAs without an element, and sizes that are not a multiple of a CTA's 256 threads
    rng = np.random.default_rng(2)
    for n in (1, 255, 64 * 256 - 1, 64 * 256 + 3, 100_003):
        v = torch.from_numpy(rng.standard_normal(n).astype(np.float32)).cuda()
        B.st_argmax_static(v, n, got, stream)
        torch.cuda.synchronize()
        assert int(got.item()) == int(np.argmax(v.cpu().numpy())), n
    # the property the entry point exists for: a call allocates no device memory and launches exactly one kernel
    torch.cuda.synchronize()
    free_before, launches_before = torch.cuda.mem_get_info()[0], B.st_kernel_launches()
    B.st_argmax_static(flat, 4096, got, stream)
    torch.cuda.synchronize()
    assert torch.cuda.mem_get_info()[0] == free_before
    assert B.st_kernel_launches() == launches_before + 1
    # sizes beyond the built-in scratch limit are refused
    with pytest.raises(B.StError) as e:
        B.st_argmax_static(flat, (1 << 22) + 1, got, stream)
    assert e.value.status == B.ST_ERR_CAPACITY
    m.close()
