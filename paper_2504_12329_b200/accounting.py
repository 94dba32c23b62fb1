"""The paper's own accounting of a Speculative Thinking run (host arithmetic on the logs a generation returns; no
part of the decode path).

* modify ratio (Table "Large Reasoning Models Monitor Small Reasoning Models"): the share of output tokens that
  come from the target model.
* FLOPs (appendix "Computation of FLOPs", as printed: no layer count, no LM head), s = sequence length, h = hidden
  size, h' = FFN size, n = attention heads:
      prefill(s) = 8 s h^2 + 16 s h + 4 s^2 h + 4 s^2 n + 6 s h h' + 2 s h'
      decode(s)  = 8 h^2 + 16 h + 4 s h + 4 s n + 6 h h' + 2 h'
* estimated speed (Eq. "Estimated Speed"): tokens / ((prefill + prefix + decode FLOPs) / capacity) with the paper's
  assumption that a prefix pass of any length costs one decode pass, and its capacity constant 3.12e10 FLOP/s.
"""
from __future__ import annotations

import numpy as np

PAPER_CAPACITY = 3.12e10


def modify_ratio(source) -> float:
    src = np.asarray(source)
    return float((src == 1).sum()) / max(1, src.size)


def _coeffs(shape):
    h, hp, n = float(shape["hidden"]), float(shape["ffn"]), float(shape["n_q_heads"])
    return h, hp, n


def flops_prefill(s, shape) -> float:
    h, hp, n = _coeffs(shape)
    s = float(s)
    return 8 * s * h * h + 16 * s * h + 4 * s * s * h + 4 * s * s * n + 6 * s * h * hp + 2 * s * hp


def flops_decode(s, shape):
    h, hp, n = _coeffs(shape)
    s = np.asarray(s, dtype=np.float64)
    return 8 * h * h + 16 * h + 4 * s * h + 4 * s * n + 6 * h * hp + 2 * hp


def flops_plain_decode(prompt_len: int, n_new: int, shape) -> float:
    """prefill(p) + sum_{i < d} decode(p + i), the sum in closed form."""
    h, hp, n = _coeffs(shape)
    p, d = float(prompt_len), float(n_new)
    const = 8 * h * h + 16 * h + 6 * h * hp + 2 * hp
    return flops_prefill(p, shape) + d * const + (4 * h + 4 * n) * (d * p + d * (d - 1) / 2)


def estimated_speed(result, prompt_len: int, small_shape, large_shape=None, capacity: float = PAPER_CAPACITY) -> float:
    """Tokens per second by the paper's estimate for one generation (log of st_generate_spec): the first pass of the
    speculative model is the prompt prefill, every other pass -- decode step or catch-up of any length -- costs
    decode(s) of the emitting model at the context s it ends on.  Valid for the one-token probe (no rollback)."""
    src = np.asarray(result.emission_source)
    fed = np.asarray(result.emission_fed)
    kv = [0, 0]
    total = 0.0
    first_small = True
    for a, m in zip(src.tolist(), fed.tolist()):
        kv[a] += m
        shape = large_shape if a == 1 else small_shape
        if a == 0 and first_small:
            total += flops_prefill(kv[0], shape)
            first_small = False
        else:
            total += float(flops_decode(kv[a], shape))
    return len(result.tokens) / (total / capacity) if total > 0 else 0.0
