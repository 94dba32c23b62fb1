"""Pins for the oracle's handoff state machine: hand-traced streams and invariants (CPU only)."""
import os

import numpy as np
import pytest

from paper_2504_12329_b200 import workloads as W

HERE = os.path.dirname(os.path.abspath(__file__))


def _trace(name):
    out = {}
    with open(os.path.join(HERE, "golden", name)) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            k, v = line.split("=")
            if k == "handoff_kinds":
                out[k] = [int(x) for x in v.split(",")]
            elif k == "handoffs":
                out[k] = [tuple(int(x) for x in h.split(":")) for h in v.split(",")]
            elif "," in v:
                out[k] = [int(x) for x in v.split(",")]
            else:
                out[k] = int(v)
    return out


LIST_PARAMS = ("keyword_ids", "affirmation_ids", "verification_ids", "aux_ids", "delimiter_ids")
RULE_TRACES = ["handoff_trace_verify_in_probe.txt", "handoff_trace_counter_reset.txt", "handoff_trace_probe_cut_replace.txt",
               "handoff_trace_probe_cut_keep.txt", "handoff_trace_delimiter_in_probe.txt", "handoff_trace_target_verification.txt",
               "handoff_trace_delimiter_set.txt"]


def load_rule_trace(name):
    """A self-describing hand-traced stream: `p.<name>=` lines are the rule parameters, the rest the expected logs."""
    T, params = {}, {}
    with open(os.path.join(HERE, "golden", name)) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            k, v = line.split("=")
            if k.startswith("p."):
                k = k[2:]
                params[k] = [int(x) for x in v.split(",")] if k in LIST_PARAMS else int(v)
            elif k == "handoffs":
                T[k] = [tuple(int(x) for x in h.split(":")) for h in v.split(",")]
            elif k in ("max_new", "kv_len_small", "kv_len_large", "budget", "budget_steps"):
                T[k] = int(v)
            else:
                T[k] = [int(x) for x in v.split(",")]
    params.setdefault("keyword_ids", [])
    return T, params


def assert_matches_trace(r, T):
    assert r.tokens.tolist() == T["tokens"]
    assert r.source.tolist() == T["source"]
    assert r.handoffs == T["handoffs"] and r.handoff_kinds == T["handoff_kinds"]
    assert r.emission_tokens.tolist() == T["force"]
    assert r.emission_source.tolist() == T["emission_source"]
    assert r.emission_fed.tolist() == T["emission_fed"]
    assert (r.kv_len_small, r.kv_len_large) == (T["kv_len_small"], T["kv_len_large"])


@pytest.fixture(scope="module")
def tiny(oracle):
    cfg_s = oracle.Config(**W.TINY_S.as_dict())
    cfg_l = oracle.Config(**W.TINY_L.as_dict())
    return oracle.Model(cfg_s, 0, 0), oracle.Model(cfg_l, 0, 1)


@pytest.mark.parametrize("name,keep", [("handoff_trace_replace.txt", False), ("handoff_trace_keep.txt", True)])
def test_hand_traced_streams(oracle, tiny, name, keep):
    T = _trace(name)
    r = oracle.generate_spec(tiny[0], tiny[1], [1, 2, 3], delimiter_id=10, keyword_ids=[11, 12, 13], n1=3,
                             keep_probe=keep, max_new_tokens=12, force=T["force"])
    assert r.rc == 0
    assert r.tokens.tolist() == T["tokens"]
    assert r.source.tolist() == T["source"]
    assert r.handoffs == T["handoffs"]
    assert r.emission_source.tolist() == T["emission_source"]
    assert r.emission_fed.tolist() == T["emission_fed"]
    assert r.emission_tokens.tolist() == T["force"][: len(r.emission_tokens)]
    assert (r.kv_len_small, r.kv_len_large) == (T["kv_len_small"], T["kv_len_large"])


def test_hand_traced_stream_every_delimiter(oracle, tiny):
    T = _trace("handoff_trace_every_delimiter.txt")
    r = oracle.generate_spec(tiny[0], tiny[1], [1, 2, 3], delimiter_id=10, keyword_ids=[11, 12, 13], n1=3,
                             max_new_tokens=12, force=T["force"], takeover_every_delimiter=True, target_first_n=2)
    assert r.rc == 0
    assert r.tokens.tolist() == T["tokens"]
    assert r.source.tolist() == T["source"]
    assert r.handoffs == T["handoffs"]
    assert r.emission_source.tolist() == T["emission_source"]
    assert r.emission_fed.tolist() == T["emission_fed"]
    assert (r.kv_len_small, r.kv_len_large) == (T["kv_len_small"], T["kv_len_large"])


RULES = dict(delimiter_id=10, keyword_ids=[11, 12, 13], affirmation_ids=[14], verification_ids=[13, 15], n1=2, n2=3, n3=2,
             neg_threshold=1, aux_ids=[40, 41])


def test_hand_traced_stream_three_takeovers(oracle, tiny):
    T = _trace("handoff_trace_three_takeovers.txt")
    r = oracle.generate_spec(tiny[0], tiny[1], [1, 2, 3], max_new_tokens=15, force=T["force"], **RULES)
    assert r.rc == 0
    assert r.tokens.tolist() == T["tokens"]
    assert r.source.tolist() == T["source"]
    assert r.handoffs == T["handoffs"]
    assert r.handoff_kinds == T["handoff_kinds"]
    assert r.emission_source.tolist() == T["emission_source"]
    assert r.emission_fed.tolist() == T["emission_fed"]
    assert (r.kv_len_small, r.kv_len_large) == (T["kv_len_small"], T["kv_len_large"])


@pytest.mark.parametrize("name", RULE_TRACES)
def test_hand_traced_rule_cases(oracle, tiny, name):
    """One hand-traced stream per reading that a transcription of the rule could get wrong: cue precedence inside
    one probe sentence, the reflection counter crossing its threshold and restarting, a probe sentence cut by
    end-of-sequence or by the budget (both probe readings), a delimiter inside a probe, a verification cue in the
    target's own sentence while it owes more / fewer than n2 tokens."""
    T, params = load_rule_trace(name)
    r = oracle.generate_spec(tiny[0], tiny[1], T["prompt"], max_new_tokens=T["max_new"], force=T["force"], **params)
    assert r.rc == 0
    assert_matches_trace(r, T)
    if "budget" in T:   # the same stream without an end-of-sequence id, cut by the token budget instead
        params = dict(params, eos_id=-1)
        r = oracle.generate_spec(tiny[0], tiny[1], T["prompt"], max_new_tokens=T["budget"], force=T["force"], **params)
        assert r.rc == 0 and r.tokens.tolist() == T["budget_tokens"] and len(r.emission_tokens) == T["budget_steps"]
        assert r.handoffs == T["handoffs"] and r.source.tolist() == T["source"][:T["budget"]]


def test_three_takeovers_reduce_and_hold_invariants(oracle, tiny):
    base = dict(delimiter_id=10, keyword_ids=[11, 12, 13], n1=3)
    force = W.full_forcing(77, 400, 1024, mean_interval=5, keyword_rate=0.7)
    plain = oracle.generate_spec(tiny[0], tiny[1], [1, 2, 3], max_new_tokens=150, force=force, **base)
    # empty extra sets and a switched-off counter are the plain rule
    same = oracle.generate_spec(tiny[0], tiny[1], [1, 2, 3], max_new_tokens=150, force=force, affirmation_ids=[],
                                verification_ids=[], neg_threshold=-1, aux_ids=[40], **base)
    assert same.tokens.tolist() == plain.tokens.tolist() and same.handoffs == plain.handoffs
    assert set(plain.handoff_kinds) == {1}
    # with the counter on, every (3) follows exactly neg_threshold + 1 reflection cues of the small model since the last (3)
    r = oracle.generate_spec(tiny[0], tiny[1], [1, 2, 3], max_new_tokens=150, force=force, neg_threshold=2, n3=4,
                             aux_ids=[40, 41, 42], **base)
    assert 3 in r.handoff_kinds and r.rc == 0
    cues = 0
    hk = dict(zip([h[1] for h in r.handoffs], r.handoff_kinds))
    for t, (tok, src) in enumerate(zip(r.emission_tokens.tolist(), r.emission_source.tolist())):
        if t in hk and src == 0:
            if tok in (11, 12, 13):
                cues += 1
            if hk[t] == 3:
                assert cues == 3
                cues = 0
    src = r.source.tolist()
    toks = r.tokens.tolist()
    for (seg, step, cu), kind in zip(r.handoffs, r.handoff_kinds):
        i = seg - 3                      # index into the generated tokens
        if kind == 3 and i + 4 <= len(src):
            assert toks[i - 3:i] == [40, 41, 42] and src[i - 3:i] == [2, 2, 2]
            assert src[i:i + 4] == [1, 1, 1, 1]
    # n_steps = tokens written by a model + dropped cues
    assert len(r.emission_tokens) == sum(1 for x in src if x != 2) + sum(1 for k, h in zip(r.handoff_kinds, r.handoffs) if h[2] > 0 or k != 2)


PROBE = dict(delimiter_id=10, keyword_ids=[11, 12], affirmation_ids=[14], verification_ids=[15], n1=3, n2=4, probe_len=3)


def test_hand_traced_stream_sentence_probe(oracle, tiny):
    T = _trace("handoff_trace_sentence_probe.txt")
    r = oracle.generate_spec(tiny[0], tiny[1], [1, 2, 3], max_new_tokens=14, force=T["force"], **PROBE)
    assert r.rc == 0
    assert r.tokens.tolist() == T["tokens"]
    assert r.source.tolist() == T["source"]
    assert r.handoffs == T["handoffs"] and r.handoff_kinds == T["handoff_kinds"]
    assert r.emission_source.tolist() == T["emission_source"]
    assert r.emission_fed.tolist() == T["emission_fed"]
    assert r.emission_tokens.tolist() == T["force"]
    assert (r.kv_len_small, r.kv_len_large) == (T["kv_len_small"], T["kv_len_large"])


def test_sentence_probe_invariants(oracle, tiny):
    rng = np.random.default_rng(4)
    force = rng.choice([10, 10, 11, 12, 14, 15, 30, 31, 32, 33, 34, 35], size=900).astype(np.int32)
    for keep in (False, True):
        r = oracle.generate_spec(tiny[0], tiny[1], [1, 2, 3], max_new_tokens=200, force=force, keep_probe=keep,
                                 neg_threshold=3, n3=5, aux_ids=[40, 41], **PROBE)
        assert r.rc == 0 and {1, 2, 3} <= set(r.handoff_kinds) and len(r.tokens) == 200
        toks, src = r.tokens.tolist(), r.source.tolist()
        for (seg, step, cu), kind in zip(r.handoffs, r.handoff_kinds):
            i = seg - 3
            if cu == 0:
                continue                                     # the target extended its own segment (verification)
            back = 3 if kind == 3 else 1                      # two auxiliary tokens sit before the segment of a (3)
            if keep:
                assert src[i - back] == 0                    # the probe sentence stays, the segment follows it
            else:
                assert toks[i - back] == 10                  # the segment (or the auxiliary sentence) starts right after the delimiter
        # the speculative model's cache never runs ahead of the text, and every step is accounted for
        assert r.kv_len_small <= 3 + 200 and r.kv_len_large <= 3 + 200
    # a probe of one token is the rule with the first-token test
    one = oracle.generate_spec(tiny[0], tiny[1], [1, 2, 3], max_new_tokens=120, force=force, neg_threshold=3, n3=5, aux_ids=[40, 41],
                               **dict(PROBE, probe_len=1))
    ref = oracle.generate_spec(tiny[0], tiny[1], [1, 2, 3], max_new_tokens=120, force=force, neg_threshold=3, n3=5, aux_ids=[40, 41],
                               **{k: v for k, v in PROBE.items() if k != "probe_len"})
    assert one.tokens.tolist() == ref.tokens.tolist() and one.handoffs == ref.handoffs


def test_every_delimiter_edge_cases(oracle, tiny):
    kw = dict(delimiter_id=10, keyword_ids=[11, 12, 13], n1=2, takeover_every_delimiter=True)
    # keywords mean nothing in this mode; a delimiter written by the target or standing in the prompt hands nothing over
    r = oracle.generate_spec(tiny[0], tiny[1], [4, 10], max_new_tokens=8, force=[11, 10, 10, 21, 12, 10, 30, 31], **kw)
    assert r.source.tolist() == [0, 0, 1, 1, 0, 0, 1, 1]
    assert r.handoffs == [(4, 1, 4), (8, 5, 3)]      # the target cached 5 tokens by its second turn: it ingests positions 5..7
    # the budget ends on the delimiter: no handoff is logged for a segment that cannot start
    r = oracle.generate_spec(tiny[0], tiny[1], [4], max_new_tokens=2, force=[5, 10], **kw)
    assert r.handoffs == [] and r.source.tolist() == [0, 0]
    # the opening segment alone; without a target both switches are ignored
    r = oracle.generate_spec(tiny[0], tiny[1], [4], max_new_tokens=5, force=[5, 6, 7, 8, 9], delimiter_id=10, keyword_ids=[],
                             n1=2, target_first_n=3)
    assert r.source.tolist() == [1, 1, 1, 0, 0] and r.handoffs == []
    r = oracle.generate_spec(tiny[0], None, [4], max_new_tokens=4, force=[5, 10, 7, 8], target_first_n=3, **kw)
    assert r.source.tolist() == [0, 0, 0, 0] and r.handoffs == []
    # every target segment has exactly n1 tokens unless the budget cuts it
    force = W.full_forcing(5, 200, 1024, mean_interval=5, keyword_rate=0.0)
    r = oracle.generate_spec(tiny[0], tiny[1], [1, 2, 3], max_new_tokens=90, force=force, **kw)
    src = r.source.tolist()
    runs = [len(x) for x in "".join(map(str, src)).split("0") if x]
    assert len(r.handoffs) >= 5 and all(n == 2 for n in runs[:-1]) and runs[-1] <= 2
    for (seg, step, cu) in r.handoffs:
        assert r.tokens[seg - 3 - 1] == 10 and src[seg - 3 - 1] == 0     # the token before the segment is a small-model delimiter


def _run(oracle, tiny, prompt, force, n1=3, max_new=10, keep=False, eos=-1, large=True):
    return oracle.generate_spec(tiny[0], tiny[1] if large else None, prompt, delimiter_id=10,
                                keyword_ids=[11, 12, 13], n1=n1, keep_probe=keep, eos_id=eos,
                                max_new_tokens=max_new, force=force)


def test_scripted_edge_cases(oracle, tiny):
    # the delimiter is the last prompt token and the first sampled token is a keyword
    r = _run(oracle, tiny, [4, 10], [12, 30, 31, 32, 33], max_new=4)
    assert r.handoffs == [(2, 0, 2)] and r.tokens.tolist() == [30, 31, 32, 33] and r.source.tolist() == [1, 1, 1, 0]
    # a keyword without a delimiter before it does nothing
    r = _run(oracle, tiny, [4, 5], [11, 12, 13, 9], max_new=4)
    assert r.handoffs == [] and r.source.tolist() == [0, 0, 0, 0]
    # the target's own delimiter+keyword does not re-trigger inside its run, but the delimiter that ends
    # the run followed by a speculative keyword does
    r = _run(oracle, tiny, [4, 10], [11, 10, 11, 10, 12, 40, 41, 42], max_new=6)
    assert r.tokens.tolist() == [10, 11, 10, 40, 41, 42]
    assert r.source.tolist() == [1, 1, 1, 1, 1, 1]
    assert r.handoffs == [(2, 0, 2), (5, 4, 1)]          # the target only lacks the last token it wrote itself
    assert r.emission_fed.tolist() == [2, 2, 1, 1, 3, 1, 1, 1]
    # the token budget ends a run early
    r = _run(oracle, tiny, [4, 10], [11, 20, 21], max_new=2)
    assert r.tokens.tolist() == [20, 21] and r.source.tolist() == [1, 1] and r.kv_len_large == 3
    # EOS inside a run stops at once
    r = _run(oracle, tiny, [4, 10], [11, 20, 99, 21], max_new=8, eos=99)
    assert r.tokens.tolist() == [20, 99] and r.source.tolist() == [1, 1]
    # n1 = 1: control returns after a single target token
    r = _run(oracle, tiny, [4, 10], [11, 20, 21, 22], n1=1, max_new=3)
    assert r.source.tolist() == [1, 0, 0] and r.emission_fed.tolist() == [2, 2, 1, 1]


def test_no_large_model_or_no_keywords_is_plain_decode(oracle, tiny):
    prompt = W.prompt_ids(3, 8, 1024)
    force = W.forcing_schedule(5, 40, mean_interval=4, keyword_rate=0.9)
    a = _run(oracle, tiny, prompt, force, max_new=20, large=False)
    b = oracle.generate_spec(tiny[0], tiny[1], prompt, delimiter_id=10, keyword_ids=[], n1=3, max_new_tokens=20,
                             force=force)
    assert a.handoffs == [] and b.handoffs == []
    assert a.tokens.tolist() == b.tokens.tolist() and set(a.source.tolist()) == {0}
    # and equals feeding the cache by hand with greedy choices
    kv = oracle.KV(tiny[0], 64)
    z = kv.forward(prompt)
    out = []
    for t in range(20):
        tok = int(force[t]) if force[t] >= 0 else oracle.argmax(z)[0]
        out.append(tok)
        z = kv.forward([tok])
    assert out == a.tokens.tolist()


@pytest.mark.parametrize("keep", [False, True])
@pytest.mark.parametrize("n1", [1, 4, 20])
def test_invariants_under_random_schedules(oracle, tiny, keep, n1):
    prompt = W.prompt_ids(100, 32, 1024)
    force = W.forcing_schedule(101 + n1, 300, mean_interval=8, keyword_rate=0.5)
    r = oracle.generate_spec(tiny[0], tiny[1], prompt, delimiter_id=10, keyword_ids=[11, 12, 13], n1=n1,
                             keep_probe=keep, max_new_tokens=128, force=force)
    assert r.rc == 0 and len(r.tokens) == 128 and len(r.handoffs) >= 2
    n_steps = len(r.emission_tokens)
    assert n_steps == (128 if keep else 128 + len(r.handoffs))
    seq = np.concatenate([prompt, r.tokens])
    src = r.source
    for seg_start, step, catch in r.handoffs:
        i = seg_start - 32                                   # index into generated tokens
        if keep:
            assert seq[seg_start - 2] == 10 and seq[seg_start - 1] in (11, 12, 13) and src[i - 1] == 0
        else:
            assert seq[seg_start - 1] == 10
        run = src[i:i + n1]
        assert np.all(run == 1)                              # the target writes exactly n1 tokens ...
        if i + n1 < 128:
            assert src[i + n1] == 0                          # ... then the speculative model resumes
        assert r.emission_source[step] == 0 and r.emission_tokens[step] in (11, 12, 13)
        assert catch >= 0
    # every target token belongs to some run
    assert src.sum() == sum(min(n1, 128 - (s - 32)) for s, _, _ in r.handoffs)
    # each model has ingested everything before the last token it was asked to emit
    assert r.kv_len_small <= 32 + 128 and r.kv_len_large <= 32 + 128
    assert sum(r.emission_fed[r.emission_source == 0]) == r.kv_len_small
    assert sum(r.emission_fed[r.emission_source == 1]) == r.kv_len_large
    # modify ratio
    assert 0.0 < src.mean() < 1.0
