"""Host-side logic of the benchmark (CPU only): the pass mix derived from a forcing schedule equals the
oracle's routing of the same schedule, and the workload generators are deterministic."""
import os
import sys

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)

import bench  # noqa: E402
from paper_2504_12329_b200 import workloads as W  # noqa: E402


def test_schedule_stats_match_oracle_routing(oracle):
    w = W.Workload("t", W.TINY_S, W.TINY_L, 24, 200, 8.0, 0.5)
    prompt, force = W.workload_inputs(w)
    # every step forced, so that routing is independent of the logits (the replay treats unforced steps as ordinary tokens)
    filled = np.where(force >= 0, force, 500).astype(np.int32)
    ts = oracle.Model(oracle.Config(**W.TINY_S.as_dict()), 0, 0)
    tl = oracle.Model(oracle.Config(**W.TINY_L.as_dict()), 0, 1)
    r = oracle.generate_spec(ts, tl, prompt, delimiter_id=W.DELIMITER_ID, keyword_ids=W.KEYWORD_IDS, n1=W.N1,
                             max_new_tokens=w.max_new_tokens, force=filled)
    stats = bench.schedule_stats(w)
    assert stats["n_tokens"] == len(r.tokens) == 200
    assert stats["steps_small"] == int((r.emission_source == 0).sum())
    assert stats["steps_large"] == int((r.emission_source == 1).sum())
    assert stats["steps_large"] == int(r.source.sum())


def test_workload_generators_are_seeded_and_shaped():
    a, fa = W.workload_inputs(W.CONFIGS["qwen1p5b_32b"])
    b, fb = W.workload_inputs(W.CONFIGS["qwen1p5b_32b"])
    assert np.array_equal(a, b) and np.array_equal(fa, fb)
    assert a.size == 256 and a.min() >= 0 and a.max() < 151936
    gaps = np.diff(np.flatnonzero(fa == W.DELIMITER_ID))
    assert 30 < gaps.mean() < 55                          # geometric, mean 40 (+1 after a keyword)
    kw = np.isin(fa, W.KEYWORD_IDS).sum() / (fa == W.DELIMITER_ID).sum()
    assert 0.2 < kw < 0.4                                 # keyword after ~30 % of the delimiters
    prompts, budgets, forces = W.batch_inputs(1, 64, 151936)
    assert len(prompts) == 64 and all(64 <= len(p) <= 512 for p in prompts)
    assert all(1024 <= x <= 8192 for x in budgets) and len(forces[0]) == 2 * budgets[0]
    # live KV of the batched workload fits beside the weights (68.6 GB) in 180 GB
    live_tokens = sum(len(p) + x for p, x in zip(prompts, budgets))
    assert live_tokens * (W.QWEN_32B.kv_bytes_per_token + W.QWEN_1P5B.kv_bytes_per_token) < 100e9


def test_streamed_bytes_match_the_shape_tables():
    assert abs(W.QWEN_1P5B.n_params_streamed * 2 / 1e9 - 3.087) < 0.01
    assert abs(W.QWEN_7B.n_params_streamed * 2 / 1e9 - 14.14) < 0.02
    assert abs(W.QWEN_32B.n_params_streamed * 2 / 1e9 - 63.97) < 0.03
    assert W.QWEN_32B.kv_bytes_per_token == 256 * 1024 and W.QWEN_1P5B.kv_bytes_per_token == 28 * 1024
