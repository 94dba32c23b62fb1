"""The paper's accounting (modify ratio, FLOP model, estimated speed): the package's closed forms against the
term-by-term restatement, and both against figures the paper prints (CPU only)."""
import types

import numpy as np
import pytest

from oracle import accounting as OA
from paper_2504_12329_b200 import accounting as A
from paper_2504_12329_b200 import workloads as W

SHAPES = {"1.5B": W.QWEN_1P5B.as_dict(), "7B": W.QWEN_7B.as_dict(), "32B": W.QWEN_32B.as_dict()}


@pytest.mark.parametrize("name", ["1.5B", "7B", "32B"])
def test_closed_form_equals_the_sum(name):
    sh = SHAPES[name]
    h, hp, n = sh["hidden"], sh["ffn"], sh["n_q_heads"]
    for p, d in [(1, 1), (37, 250), (256, 2048)]:
        want = OA.flops_total(p, d, h, hp, n)
        assert A.flops_plain_decode(p, d, sh) == pytest.approx(want, rel=1e-12)
        assert float(A.flops_decode(p, sh)) == OA.flops_decode(p, h, hp, n)
        assert A.flops_prefill(p, sh) == OA.flops_prefill(p, h, hp, n)
    # prefill of one token is a decode step at context 1
    assert A.flops_prefill(1, sh) == float(A.flops_decode(1, sh))


# MATH500 rows of the paper's results table: average output length and estimated speed of each model alone.  The
# prompt lengths and the per-problem averaging are not printed, so the pin is loose (prompt assumed 100 tokens).
@pytest.mark.parametrize("name,avg_len,printed", [("1.5B", 5439, 242.6), ("7B", 3802, 63.7), ("32B", 3802, 32.2)])
def test_estimated_speed_against_the_printed_table(name, avg_len, printed):
    sh = SHAPES[name]
    got = avg_len / (A.flops_plain_decode(100, avg_len, sh) / A.PAPER_CAPACITY)
    assert got == pytest.approx(OA.estimated_speed_plain(100, avg_len, sh["hidden"], sh["ffn"], sh["n_q_heads"]), rel=1e-12)
    assert got == pytest.approx(printed, rel=0.16)


def test_estimated_speed_of_a_logged_run_and_modify_ratio():
    # the hand-traced stream of the handoff rule (tests/golden/handoff_trace_replace.txt): modify ratio 6 / 12
    src = [0, 0, 1, 1, 1, 0, 0, 0, 0, 1, 1, 1]
    assert A.modify_ratio(src) == OA.modify_ratio(src) == 0.5
    r = types.SimpleNamespace(tokens=np.arange(12), emission_source=np.array([0, 0, 0, 1, 1, 1, 0, 0, 0, 0, 0, 1, 1, 1]),
                              emission_fed=np.array([3, 1, 1, 5, 1, 1, 3, 1, 1, 1, 1, 5, 1, 1]))
    S, L = SHAPES["1.5B"], SHAPES["32B"]
    s_args, l_args = (S["hidden"], S["ffn"], S["n_q_heads"]), (L["hidden"], L["ffn"], L["n_q_heads"])
    total = OA.flops_prefill(3, *s_args)
    ctx_small, ctx_large = [4, 5, 8, 9, 10, 11, 12], [5, 6, 7, 12, 13, 14]     # context each later pass ends on
    total += sum(OA.flops_decode(c, *s_args) for c in ctx_small) + sum(OA.flops_decode(c, *l_args) for c in ctx_large)
    assert A.estimated_speed(r, 3, S, L) == pytest.approx(12 / (total / 3.12e10), rel=1e-12)
    # a run without the target is the plain formula
    plain = types.SimpleNamespace(tokens=np.arange(50), emission_source=np.zeros(50, int), emission_fed=np.array([20] + [1] * 49))
    assert A.estimated_speed(plain, 20, S) == pytest.approx(OA.estimated_speed_plain(20, 50, *s_args) * 1.0, rel=0.03)
