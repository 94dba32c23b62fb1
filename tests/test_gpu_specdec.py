"""GPU parity of greedy speculative decoding (the paper's comparison system) against the CPU oracle and against a
hand-traced stream, through the C ABI."""
import numpy as np
import pytest

from paper_2504_12329_b200 import workloads as W
from parity_utils import MARGIN, shape_dict
from test_oracle_specdec import assert_matches_specdec_trace, load_specdec_trace

pytestmark = pytest.mark.gpu

torch = pytest.importorskip("torch")


@pytest.fixture(scope="module")
def B():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2504_12329_b200 import binding, build
    build.build()
    binding.lib()
    return binding


def _mixed_drafts(want, gamma, vocab, seed, p_good=0.7):
    """Drafts that agree with the target's stream `want` with probability p_good: replays the rounds to know which
    generated position each draft stands for."""
    rng = np.random.default_rng(seed)
    n, pos, fd = len(want), 0, []
    while pos < n:
        g = min(gamma, n - pos - 1)
        alive, nacc = True, 0
        for i in range(g):
            good = rng.random() < p_good
            fd.append(int(want[pos + i]) if good else int((want[pos + i] + 1 + rng.integers(0, 5)) % vocab))
            if alive and good:
                nacc += 1
            else:
                alive = False
        pos += nacc + 1
    return np.asarray(fd, dtype=np.int32)


def _compare(want, got):
    """Tokens, sources and rounds must agree as long as every decision of the target so far was clear in the oracle
    (top-2 margin of its logits row at least MARGIN); returns how many generated positions were compared."""
    low = np.nonzero(want.choice_margin < MARGIN)[0]
    n_ok = int(low[0]) if len(low) else len(want.tokens)
    assert got.tokens[:n_ok].tolist() == want.tokens[:n_ok].tolist()
    assert got.source[:n_ok].tolist() == want.source[:n_ok].tolist()
    # rounds that lie entirely inside the compared prefix
    done, k = 0, 0
    for (d, a) in want.rounds:
        if done + a + 1 > n_ok:
            break
        assert got.rounds[k] == (d, a), (k, got.rounds[k], (d, a))
        done += a + 1
        k += 1
    if n_ok == len(want.tokens):
        assert got.rounds == want.rounds
        assert (got.kv_len_small, got.kv_len_large) == (want.kv_len_small, want.kv_len_large)
        assert (got.n_drafted, got.n_accepted) == (want.n_drafted, want.n_accepted)
    return n_ok


def test_hand_traced_stream_on_device(B):
    T = load_specdec_trace()
    gs = B.Model(shape_dict(W.TINY_S), seed=0, tag=0, max_tokens=256)
    gl = B.Model(shape_dict(W.TINY_L), seed=0, tag=1, max_tokens=256)
    for _ in range(2):   # a second call on the same models starts from clean caches
        r = B.st_generate_specdec(gs, gl, T["prompt"], gamma=T["gamma"], max_new_tokens=T["max_new"],
                                  force_draft=T["force_draft"], force_target=T["force_target"])
        assert_matches_specdec_trace(r, T)
        assert r.draft_tokens.tolist() == T["force_draft"]
    # edges: a budget of one token (no draft), end-of-sequence among the accepted drafts
    r = B.st_generate_specdec(gs, gl, [4, 5, 6], gamma=5, max_new_tokens=1, force_target=[9])
    assert r.tokens.tolist() == [9] and r.rounds == [(0, 0)] and (r.kv_len_small, r.kv_len_large) == (0, 3)
    r = B.st_generate_specdec(gs, gl, [4, 5, 6], gamma=3, max_new_tokens=9, eos_id=7, force_draft=[5, 7, 8], force_target=[5, 7, 8, 9])
    assert r.tokens.tolist() == [5, 7] and r.rounds == [(3, 3)]
    assert gs.st_last_device_status() == 0 and gl.st_last_device_status() == 0
    gs.close()
    gl.close()


@pytest.mark.parametrize("gamma", [4, 20])
def test_tiny_pair_against_oracle(B, oracle, gamma):
    S, L = shape_dict(W.TINY_S), shape_dict(W.TINY_L)
    os_, ol = oracle.Model(oracle.Config(**S), 0, 0), oracle.Model(oracle.Config(**L), 0, 1)
    gs = B.Model(S, seed=0, tag=0, max_tokens=1024)
    gl = B.Model(L, seed=0, tag=1, max_tokens=1024)
    prompt = W.prompt_ids(41, 300, 1024)   # longer than one pass: the target ingests it in chunks before it scores
    n = 90
    free = oracle.generate_specdec(os_, ol, prompt, gamma=gamma, max_new_tokens=n)
    fd = _mixed_drafts(free.tokens, gamma, 1024, 5)
    want = oracle.generate_specdec(os_, ol, prompt, gamma=gamma, max_new_tokens=n, force_draft=fd)
    assert want.rc == 0 and want.tokens.tolist() == free.tokens.tolist()       # the output is the target's own continuation
    assert 0 < want.n_accepted < want.n_drafted
    got = B.st_generate_specdec(gs, gl, prompt, gamma=gamma, max_new_tokens=n, force_draft=fd)
    n_ok = _compare(want, got)
    # fully forced on both sides: every log bit-exact whatever the margins
    want2 = oracle.generate_specdec(os_, ol, prompt, gamma=gamma, max_new_tokens=n, force_draft=fd, force_target=free.tokens)
    got2 = B.st_generate_specdec(gs, gl, prompt, gamma=gamma, max_new_tokens=n, force_draft=fd, force_target=free.tokens)
    assert got2.tokens.tolist() == want2.tokens.tolist() and got2.rounds == want2.rounds and got2.source.tolist() == want2.source.tolist()
    assert (got2.kv_len_small, got2.kv_len_large) == (want2.kv_len_small, want2.kv_len_large)
    # the target's greedy choices behind the forced stream agree with the oracle's wherever its margin is clear
    clear = want2.choice_margin >= MARGIN
    assert clear.sum() >= 10
    # unforced drafts: the speculative model's own choices, compared through the draft log
    got3 = B.st_generate_specdec(gs, gl, prompt, gamma=gamma, max_new_tokens=30, force_target=free.tokens)
    want3 = oracle.generate_specdec(os_, ol, prompt, gamma=gamma, max_new_tokens=30, force_target=free.tokens)
    low = np.nonzero(want3.draft_margin < MARGIN)[0]
    k_ok = int(low[0]) if len(low) else len(want3.draft_margin)
    assert got3.draft_tokens[:k_ok].tolist() == [int(x) for x in got3.draft_argmax[:k_ok]]
    print(f"gamma {gamma}: {n_ok} of {n} positions compared free-running, {int(clear.sum())} clear target choices, {k_ok} drafts compared")
    assert gs.st_last_device_status() == 0 and gl.st_last_device_status() == 0
    gs.close()
    gl.close()


def test_7b_32b_two_layer_cuts(B, oracle):
    """The paper's pair for this comparison (7B speculative, 32B target; equal vocabularies), two layers deep with the
    vocabulary cut so that the oracle finishes in seconds; 20 drafts per round as in the paper."""
    S = shape_dict(W.QWEN_7B, n_layers=2, vocab=4096)
    L = shape_dict(W.QWEN_32B, n_layers=2, vocab=4096)
    os_, ol = oracle.Model(oracle.Config(**S), 0, 0), oracle.Model(oracle.Config(**L), 0, 1)
    gs = B.Model(S, seed=0, tag=0, max_tokens=512)
    gl = B.Model(L, seed=0, tag=1, max_tokens=512)
    prompt = W.prompt_ids(43, 24, 4096)
    n = 44
    free = oracle.generate_specdec(os_, ol, prompt, gamma=20, max_new_tokens=n)
    fd = _mixed_drafts(free.tokens, 20, 4096, 6, p_good=0.85)
    want = oracle.generate_specdec(os_, ol, prompt, gamma=20, max_new_tokens=n, force_draft=fd, force_target=free.tokens)
    got = B.st_generate_specdec(gs, gl, prompt, gamma=20, max_new_tokens=n, force_draft=fd, force_target=free.tokens)
    assert got.tokens.tolist() == want.tokens.tolist() and got.rounds == want.rounds
    assert (got.kv_len_small, got.kv_len_large) == (want.kv_len_small, want.kv_len_large)
    # the target's own greedy choices (before forcing) against the oracle's stream, where the oracle's margin is clear
    clear = want.choice_margin >= MARGIN
    assert clear.sum() >= 5
    assert got.choice_argmax[clear].tolist() == free.tokens[clear].tolist()
    assert gs.st_last_device_status() == 0 and gl.st_last_device_status() == 0
    gs.close()
    gl.close()


def test_bounded_waits_expire_without_hanging(B, monkeypatch):
    """Every device-side wait has a poll limit.  The self-test makes two of them run out (an mbarrier nobody arms,
    the decode kernel's grid barrier without the other arrivals): the kernel must return, the call must report
    ST_ERR_TIMEOUT, and the same model must work normally afterwards.  The generation loop's pass bound is made to
    run out the same way.  Nothing here traps, faults or spins without a limit."""
    S, L = shape_dict(W.TINY_S), shape_dict(W.TINY_L)
    gs = B.Model(S, seed=0, tag=0, max_tokens=512)
    gl = B.Model(L, seed=0, tag=1, max_tokens=512)
    prompt = W.prompt_ids(100, 32, 1024)
    force = W.full_forcing(101, 200, 1024, mean_interval=8, keyword_rate=0.5)
    kw = dict(delimiter_id=W.DELIMITER_ID, keyword_ids=W.KEYWORD_IDS, n1=4, max_new_tokens=40, force=force)
    ref = B.st_generate_spec(gs, gl, prompt, **kw)
    for which in (0, 1):
        assert gs.st_selftest_bounded_wait(which) == B.ST_ERR_TIMEOUT
        assert gs.st_last_device_status() == 0
        again = B.st_generate_spec(gs, gl, prompt, **kw)
        assert again.tokens.tolist() == ref.tokens.tolist() and again.handoffs == ref.handoffs
    # the device loop's bound on passes: two passes, then the loop ends with the status bit set
    monkeypatch.setenv("ST_TEST_PASS_CAP", "2")
    with pytest.raises(B.StError) as e:
        B.st_generate_spec(gs, gl, prompt, **kw)
    assert e.value.status == B.ST_ERR_TIMEOUT
    monkeypatch.delenv("ST_TEST_PASS_CAP")
    again = B.st_generate_spec(gs, gl, prompt, **kw)
    assert again.tokens.tolist() == ref.tokens.tolist()
    gs.close()
    gl.close()
