"""Pins for the oracle's greedy speculative decoding (the paper's comparison system): a hand-traced stream and
the invariants of the published algorithm (CPU only)."""
import os

import numpy as np
import pytest

from paper_2504_12329_b200 import workloads as W

HERE = os.path.dirname(os.path.abspath(__file__))


def load_specdec_trace(name="specdec_trace.txt"):
    T = {}
    with open(os.path.join(HERE, "golden", name)) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            k, v = line.split("=")
            if k == "rounds":
                T[k] = [tuple(int(x) for x in r.split(":")) for r in v.split(",")]
            elif k in ("gamma", "max_new", "kv_len_small", "kv_len_large"):
                T[k] = int(v)
            else:
                T[k] = [int(x) for x in v.split(",")]
    return T


def assert_matches_specdec_trace(r, T):
    assert r.tokens.tolist() == T["tokens"]
    assert r.source.tolist() == T["source"]
    assert r.rounds == T["rounds"]
    assert (r.kv_len_small, r.kv_len_large) == (T["kv_len_small"], T["kv_len_large"])
    assert r.n_drafted == sum(d for d, _ in T["rounds"]) and r.n_accepted == sum(a for _, a in T["rounds"])


@pytest.fixture(scope="module")
def tiny(oracle):
    return (oracle.Model(oracle.Config(**W.TINY_S.as_dict()), 0, 0), oracle.Model(oracle.Config(**W.TINY_L.as_dict()), 0, 1))


def _greedy(oracle, model, prompt, n):
    kv = oracle.KV(model, len(prompt) + n + 1)
    z = kv.forward(prompt)
    out = []
    for _ in range(n):
        tok = oracle.argmax(z)[0]
        out.append(tok)
        z = kv.forward([tok])
    return out


def test_hand_traced_stream(oracle, tiny):
    T = load_specdec_trace()
    r = oracle.generate_specdec(tiny[0], tiny[1], T["prompt"], gamma=T["gamma"], max_new_tokens=T["max_new"],
                                force_draft=T["force_draft"], force_target=T["force_target"])
    assert r.rc == 0
    assert_matches_specdec_trace(r, T)


def test_output_is_the_targets_own_greedy_continuation(oracle, tiny):
    """Whatever the speculative model drafts, greedy speculative decoding writes exactly what the target would have
    written alone -- here against a plain cached decode loop of the target, for a different draft model (almost every
    draft rejected), for forced drafts, and for the target drafting for itself (every draft accepted)."""
    prompt = W.prompt_ids(3, 9, 1024)
    want = _greedy(oracle, tiny[1], prompt, 25)
    for gamma in (1, 4, 20):
        r = oracle.generate_specdec(tiny[0], tiny[1], prompt, gamma=gamma, max_new_tokens=25)
        assert r.rc == 0 and r.tokens.tolist() == want
        assert sum(a + 1 for _, a in r.rounds) == 25 and all(a <= d <= gamma for d, a in r.rounds)
        assert r.kv_len_large == len(prompt) + 24 and r.kv_len_small <= len(prompt) + 24
    # drafts taken from the target's own stream at some positions: they are accepted exactly where they stand
    forced = np.full(60, -1, dtype=np.int32)
    r0 = oracle.generate_specdec(tiny[0], tiny[1], prompt, gamma=4, max_new_tokens=25, force_draft=forced)
    assert r0.tokens.tolist() == want
    same = oracle.generate_specdec(tiny[1], tiny[1], prompt, gamma=4, max_new_tokens=25)
    assert same.tokens.tolist() == want
    assert same.rounds == [(4, 4)] * 5 and same.n_accepted == same.n_drafted == 20
    assert same.source.tolist() == ([0, 0, 0, 0, 1] * 5)


def test_budget_eos_and_forcing_edges(oracle, tiny):
    prompt = [4, 5, 6]
    # a budget of one token: no draft at all
    r = oracle.generate_specdec(tiny[0], tiny[1], prompt, gamma=5, max_new_tokens=1, force_target=[9])
    assert r.tokens.tolist() == [9] and r.rounds == [(0, 0)] and r.source.tolist() == [1]
    assert (r.kv_len_small, r.kv_len_large) == (0, 3)
    # end-of-sequence among the accepted drafts ends the output there
    r = oracle.generate_specdec(tiny[0], tiny[1], prompt, gamma=3, max_new_tokens=9, eos_id=7,
                                force_draft=[5, 7, 8], force_target=[5, 7, 8, 9])
    assert r.tokens.tolist() == [5, 7] and r.rounds == [(3, 3)]
    # ... and as the target's own token
    r = oracle.generate_specdec(tiny[0], tiny[1], prompt, gamma=2, max_new_tokens=9, eos_id=7,
                                force_draft=[5, 6], force_target=[5, 7])
    assert r.tokens.tolist() == [5, 7] and r.rounds == [(2, 1)] and r.source.tolist() == [0, 1]
    # rejection rate of a forced stream: every second round loses its last draft
    ft = list(range(100, 130))
    fd = []
    for k in range(0, 30, 3):            # gamma = 2 -> rounds of up to 3 tokens
        fd += [ft[k], ft[k + 1] if (k // 3) % 2 == 0 else 0]
    r = oracle.generate_specdec(tiny[0], tiny[1], prompt, gamma=2, max_new_tokens=12, force_draft=fd, force_target=ft)
    assert r.tokens.tolist() == ft[:12]
    assert r.rounds[0] == (2, 2) and r.rounds[1][1] in (0, 1)
