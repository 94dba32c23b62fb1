"""GPU parity: the CUDA library (through its C ABI) against the CPU oracle, element by element."""
import numpy as np
import pytest

from paper_2504_12329_b200 import workloads as W
from parity_utils import MARGIN, assert_logits_close, shape_dict

pytestmark = pytest.mark.gpu

torch = pytest.importorskip("torch")


@pytest.fixture(scope="module")
def B():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2504_12329_b200 import binding, build
    build.build()   # no-op when the in-tree library is newer than its sources
    binding.lib()
    return binding


def test_seeded_weights_bit_identical(B, oracle):
    for seed, tag, tid, idx0, n in [(0, 0, 0, 0, 100_003), (0, 1, 17, 0, 4096), (5, 2, 16 * 64 + 11, 123_456_789_012, 70_001),
                                    (0, 0, 1, (1 << 33) + 5, 999)]:
        out = torch.empty(n, dtype=torch.int16, device="cuda")
        B.st_fill_tensor_bf16(seed, tag, tid, idx0, n, out)
        torch.cuda.synchronize()
        got = out.cpu().numpy().view(np.uint16)
        want = (oracle.fill_tensor(seed, tag, tid, idx0, n).view(np.uint32) >> 16).astype(np.uint16)
        assert np.array_equal(got, want)


def _teacher_forced(B, oracle, shape, seed, tag, chunks, n_decode, page_size=64, tok_seed=3):
    """Prefill in the given chunks, then n_decode single steps, all tokens given; compare every logits row."""
    rng = np.random.default_rng(tok_seed)
    total = sum(chunks) + n_decode
    tokens = rng.integers(0, shape["vocab"], size=total).astype(np.int32)
    om = oracle.Model(oracle.Config(**shape), seed, tag)
    okv = oracle.KV(om, total + 1)
    gm = B.Model(shape, seed=seed, tag=tag, max_seqs=2, max_tokens=2 * total + 64, page_size=page_size)
    slot = gm.st_seq_alloc()
    logits = torch.empty(shape["vocab"], dtype=torch.float32, device="cuda")
    worst = (0.0, 1.0)
    i = 0
    for c in chunks:
        want = okv.forward(tokens[i:i + c])
        gm.st_prefill(slot, tokens[i:i + c], logits)
        torch.cuda.synchronize()
        e, cs = assert_logits_close(logits.cpu().numpy(), want, f"prefill chunk at {i} (+{c})")
        worst = (max(worst[0], e), min(worst[1], cs))
        i += c
        assert gm.st_kv_len(slot) == i
    tok_dev = torch.empty(1, dtype=torch.int32, device="cuda")
    amax = torch.empty(1, dtype=torch.int32, device="cuda")
    for _ in range(n_decode):
        want = okv.forward(tokens[i:i + 1])
        tok_dev.copy_(torch.from_numpy(tokens[i:i + 1]))
        gm.st_decode_step([slot], tok_dev, logits, amax)
        torch.cuda.synchronize()
        got = logits.cpu().numpy()
        e, cs = assert_logits_close(got, want, f"decode at {i}")
        worst = (max(worst[0], e), min(worst[1], cs))
        gi, margin = oracle.argmax(want)
        if margin >= MARGIN:
            assert int(amax.item()) == gi
        assert int(amax.item()) == int(np.argmax(got))       # lowest-id argmax of its own logits
        i += 1
    assert gm.st_last_device_status() == 0
    gm.close()
    print(f"{shape['hidden']}x{shape['n_layers']}: worst max-abs {worst[0]:.4f}, worst cosine {worst[1]:.7f}")
    return worst


@pytest.mark.parametrize("shape,tag", [(W.TINY_S, 0), (W.TINY_L, 1)])
@pytest.mark.parametrize("page_size", [16, 64])
def test_tiny_models_teacher_forced(B, oracle, shape, tag, page_size):
    # chunk sizes span one row, a ragged tile, several tiles and a page boundary
    _teacher_forced(B, oracle, shape_dict(shape), 0, tag, chunks=[1, 2, 37, 65, 130], n_decode=20, page_size=page_size)


def test_decode_from_empty_cache_and_long_context(B, oracle):
    # first token through the decode path, then enough context to use several key splits
    _teacher_forced(B, oracle, shape_dict(W.TINY_S), 1, 0, chunks=[1], n_decode=3)
    _teacher_forced(B, oracle, shape_dict(W.TINY_S), 1, 0, chunks=[700], n_decode=4)


@pytest.mark.parametrize("shape", [W.QWEN_1P5B, W.QWEN_7B, W.QWEN_32B])
def test_full_width_two_layers(B, oracle, shape):
    """Full hidden/FFN/vocabulary widths of the large shapes (so every kernel runs in the launch
    configuration the full model uses), two layers deep so that the oracle finishes in seconds."""
    _teacher_forced(B, oracle, shape_dict(shape, n_layers=2), 0, 3, chunks=[19], n_decode=3)


@pytest.mark.parametrize("shape", [W.QWEN_1P5B, W.QWEN_32B])
def test_full_width_two_layers_longer_context(B, oracle, shape):
    """head_dim 128 with a context that needs several key splits and K/V pages in the decode kernel (the splits'
    first keys are not multiples of the staging box), a catch-up sized chunk over that context (multi-row
    attention with key splits) and a 256-row prompt chunk; vocabulary cut to keep the oracle fast."""
    _teacher_forced(B, oracle, shape_dict(shape, n_layers=2, vocab=4096), 0, 3, chunks=[256, 256, 45, 20, 130], n_decode=6)


def _batched_decode(B, oracle, shape, lengths, n_steps):
    """Sequences of different cached lengths decoded together (one st_decode_step call per step, all rows through
    the tensor-core pass); every row's logits are compared with the oracle run on that sequence alone."""
    rng = np.random.default_rng(11)
    n = len(lengths)
    om = oracle.Model(oracle.Config(**shape), 0, 2)
    gm = B.Model(shape, seed=0, tag=2, max_seqs=n, max_tokens=sum(lengths) + n * (n_steps + 64))
    okvs, slots, toks = [], [], []
    for ln in lengths:
        t = rng.integers(0, shape["vocab"], size=ln + n_steps).astype(np.int32)
        okv = oracle.KV(om, ln + n_steps + 1)
        okv.forward(t[:ln])
        slot = gm.st_seq_alloc()
        for i in range(0, ln, 256):
            gm.st_prefill(slot, t[i:min(ln, i + 256)])
        okvs.append(okv)
        slots.append(slot)
        toks.append(t)
    logits = torch.empty((n, shape["vocab"]), dtype=torch.float32, device="cuda")
    amax = torch.empty(n, dtype=torch.int32, device="cuda")
    worst = 0.0
    for k in range(n_steps):
        step_toks = np.array([toks[i][lengths[i] + k] for i in range(n)], dtype=np.int32)
        gm.st_decode_step(slots, torch.from_numpy(step_toks).cuda(), logits, amax)
        torch.cuda.synchronize()
        got = logits.cpu().numpy()
        for i in range(n):
            want = okvs[i].forward(step_toks[i:i + 1])
            e, _ = assert_logits_close(got[i], want, f"step {k}, sequence {i} (cached {lengths[i] + k})")
            worst = max(worst, e)
            gi, margin = oracle.argmax(want)
            if margin >= MARGIN:
                assert int(amax[i].item()) == gi
            assert int(amax[i].item()) == int(np.argmax(got[i]))
            assert gm.st_kv_len(slots[i]) == lengths[i] + k + 1
    assert gm.st_last_device_status() == 0
    gm.close()
    return worst


def test_batched_decode_tiny(B, oracle):
    # ragged lengths: empty-ish, inside a page, page boundaries, several 128-key tiles
    _batched_decode(B, oracle, shape_dict(W.TINY_L), [1, 15, 16, 63, 64, 127, 128, 300, 517], 3)


@pytest.mark.parametrize("shape", [W.QWEN_1P5B, W.QWEN_32B])
def test_batched_decode_full_width_two_layers(B, oracle, shape):
    _batched_decode(B, oracle, shape_dict(shape, n_layers=2, vocab=4096), [5, 70, 129, 260], 2)


def test_qwen1p5b_full_depth(B, oracle):
    """All 28 layers of the 1.5B shape: prompt prefill, a catch-up sized chunk and decode steps."""
    _teacher_forced(B, oracle, shape_dict(W.QWEN_1P5B), 0, 0, chunks=[24, 20], n_decode=4)


def _gen_both(B, oracle, small_shape, large_shape, prompt, force, *, n1, keep, max_new, trace=0, eos=-1, page_size=64):
    os_ = oracle.Model(oracle.Config(**small_shape), 0, 0)
    ol = oracle.Model(oracle.Config(**large_shape), 0, 1) if large_shape else None
    want = oracle.generate_spec(os_, ol, prompt, delimiter_id=W.DELIMITER_ID, keyword_ids=W.KEYWORD_IDS, n1=n1,
                                keep_probe=keep, eos_id=eos, max_new_tokens=max_new, force=force, trace_n_steps=trace)
    cap = len(prompt) + max_new + 64
    gs = B.Model(small_shape, seed=0, tag=0, max_tokens=cap, page_size=page_size)
    gl = B.Model(large_shape, seed=0, tag=1, max_tokens=cap, page_size=page_size) if large_shape else None
    got = B.st_generate_spec(gs, gl, prompt, delimiter_id=W.DELIMITER_ID, keyword_ids=W.KEYWORD_IDS, n1=n1,
                             keep_probe=keep, eos_id=eos, max_new_tokens=max_new, force=force, trace_n_steps=trace)
    gs.close()
    if gl:
        gl.close()
    return want, got


def _assert_routing_equal(want, got):
    assert got.tokens.tolist() == want.tokens.tolist()
    assert got.source.tolist() == want.source.tolist()
    assert got.handoffs == want.handoffs
    assert got.emission_tokens.tolist() == want.emission_tokens.tolist()
    assert got.emission_source.tolist() == want.emission_source.tolist()
    assert got.emission_fed.tolist() == want.emission_fed.tolist()
    assert (got.kv_len_small, got.kv_len_large) == (want.kv_len_small, want.kv_len_large)
    assert got.n_steps == len(want.emission_tokens)


@pytest.mark.parametrize("keep", [False, True])
def test_hand_traced_stream_on_device(B, oracle, keep):
    force = [5, 10, 11, 7, 8, 9, 6, 10, 4, 10, 12, 20, 21, 22]
    want, got = _gen_both(B, oracle, shape_dict(W.TINY_S), shape_dict(W.TINY_L), [1, 2, 3], force, n1=3, keep=keep, max_new=12)
    _assert_routing_equal(want, got)
    if not keep:
        assert got.tokens.tolist() == [5, 10, 7, 8, 9, 6, 10, 4, 10, 20, 21, 22]
        assert got.handoffs == [(5, 2, 5), (12, 10, 5)]


@pytest.mark.parametrize("keep", [False, True])
@pytest.mark.parametrize("n1", [4, 20])
def test_tiny_pair_fully_forced_routing_and_logits(B, oracle, keep, n1):
    """Tiny pair, 32-token prompt, 128 tokens, every step forced: routing is bit-exact and every
    step's logits are within tolerance."""
    prompt = W.prompt_ids(100, 32, 1024)
    force = W.full_forcing(101, 300, 1024, mean_interval=8, keyword_rate=0.5)
    want, got = _gen_both(B, oracle, shape_dict(W.TINY_S), shape_dict(W.TINY_L), prompt, force, n1=n1, keep=keep,
                          max_new=128, trace=300)
    _assert_routing_equal(want, got)
    assert len(want.handoffs) >= 2
    n = len(want.emission_tokens)
    for t in range(n):
        assert_logits_close(got.logits_trace[t], want.logits_trace[t], f"step {t}")
        if want.emission_margin[t] >= MARGIN:
            assert got.emission_argmax[t] == want.emission_argmax[t]


def test_tiny_pair_free_running(B, oracle):
    """Tiny pair with the sparse schedule (delimiters/keywords forced, everything else greedy): tokens must
    match the oracle at every step whose top-2 margin is at least 0.05; after the first low-margin
    disagreement the comparison continues teacher-forced."""
    prompt = W.prompt_ids(100, 32, 1024)
    force = W.forcing_schedule(101, 300, mean_interval=8, keyword_rate=0.5)
    want, got = _gen_both(B, oracle, shape_dict(W.TINY_S), shape_dict(W.TINY_L), prompt, force, n1=4, keep=False, max_new=128)
    n = min(len(want.emission_tokens), len(got.emission_tokens))
    diverged = None
    for t in range(n):
        if got.emission_tokens[t] != want.emission_tokens[t]:
            assert want.emission_margin[t] < MARGIN, f"step {t}: tokens differ at margin {want.emission_margin[t]}"
            diverged = t
            break
    if diverged is None:
        _assert_routing_equal(want, got)
    else:
        forced = want.emission_tokens.copy()
        want2, got2 = _gen_both(B, oracle, shape_dict(W.TINY_S), shape_dict(W.TINY_L), prompt, forced, n1=4, keep=False, max_new=128)
        _assert_routing_equal(want2, got2)


def test_plain_decode_without_large_model(B, oracle):
    prompt = W.prompt_ids(7, 16, 1024)
    want, got = _gen_both(B, oracle, shape_dict(W.TINY_S), None, prompt, None, n1=20, keep=False, max_new=48, trace=48)
    assert got.handoffs == [] and set(got.source.tolist()) == {0}
    for t in range(len(want.emission_tokens)):
        assert_logits_close(got.logits_trace[t], want.logits_trace[t], f"step {t}")
        if got.emission_tokens[t] != want.emission_tokens[t]:
            assert want.emission_margin[t] < MARGIN
            break


def test_edge_cases_on_device(B, oracle):
    S, L = shape_dict(W.TINY_S), shape_dict(W.TINY_L)
    # delimiter ends the prompt; EOS inside a run; budget ends a run; n1 = 1; re-trigger; zero new tokens
    for prompt, force, kw in [([4, 10], [12, 30, 31, 32, 33], dict(n1=3, max_new=4)),
                              ([4, 10], [11, 20, 99, 21], dict(n1=3, max_new=8, eos=99)),
                              ([4, 10], [11, 20, 21], dict(n1=3, max_new=2)),
                              ([4, 10], [11, 20, 21, 22], dict(n1=1, max_new=3)),
                              ([4, 10], [11, 10, 11, 10, 12, 40, 41, 42], dict(n1=3, max_new=6)),
                              ([4], [], dict(n1=3, max_new=0))]:
        for keep in (False, True):
            want, got = _gen_both(B, oracle, S, L, prompt, force if force else None, keep=keep, **kw)
            _assert_routing_equal(want, got)


def test_host_side_errors(B):
    S = shape_dict(W.TINY_S)
    m = B.Model(S, max_tokens=128)
    with pytest.raises(B.StError) as e:
        B.st_generate_spec(m, None, [1, 2000], delimiter_id=10, keyword_ids=[11], max_new_tokens=4)
    assert e.value.status == B.ST_ERR_VOCAB
    with pytest.raises(B.StError) as e:
        B.st_generate_spec(m, None, [1, 2], delimiter_id=10, keyword_ids=[11], max_new_tokens=4000)
    assert e.value.status == B.ST_ERR_KV_FULL
    with pytest.raises(B.StError) as e:
        B.st_generate_spec(m, None, [1, 2], delimiter_id=10, keyword_ids=[11], max_new_tokens=8, cap_steps=3)
    assert e.value.status == B.ST_ERR_CAPACITY
    slot = m.st_seq_alloc()
    with pytest.raises(B.StError) as e:
        m.st_seq_alloc()
    assert e.value.status == B.ST_ERR_KV_FULL
    with pytest.raises(B.StError) as e:
        m.st_prefill(slot, [5000])
    assert e.value.status == B.ST_ERR_VOCAB
    with pytest.raises(B.StError) as e:
        m.st_prefill(slot, list(range(400)))
    assert e.value.status == B.ST_ERR_KV_FULL
    m.st_seq_free(slot)
    # the model still works after the refused calls
    r = B.st_generate_spec(m, None, [1, 2], delimiter_id=10, keyword_ids=[11], max_new_tokens=4)
    assert len(r.tokens) == 4
    bad = dict(S, head_dim=48)
    with pytest.raises(B.StError) as e:
        B.Model(bad)
    assert e.value.status == B.ST_ERR_UNSUPPORTED
    m.close()


def test_batched_ragged_sequences(B, oracle):
    """The batched entry point on the tiny pair: 6 independent sequences with ragged prompts, budgets and
    schedules (every step forced); each sequence's routing equals the oracle's run of that sequence alone."""
    S, L = shape_dict(W.TINY_S), shape_dict(W.TINY_L)
    prompts, budgets, forces = W.batch_inputs(7, 6, 1024, prompt_range=(5, 40), budget_range=(20, 90), mean_interval=6,
                                              keyword_rate=0.6)
    forces = [W.full_forcing(900 + i, len(f), 1024, mean_interval=6, keyword_rate=0.6) for i, f in enumerate(forces)]
    gs = B.Model(S, seed=0, tag=0, max_tokens=256)
    gl = B.Model(L, seed=0, tag=1, max_tokens=256)
    got = B.st_generate_spec_batch(gs, gl, prompts, delimiter_id=W.DELIMITER_ID, keyword_ids=W.KEYWORD_IDS, n1=4,
                                   max_new_tokens=budgets, forces=forces)
    os_, ol = oracle.Model(oracle.Config(**S), 0, 0), oracle.Model(oracle.Config(**L), 0, 1)
    assert len(got) == 6
    n_hand = 0
    for i in range(6):
        want = oracle.generate_spec(os_, ol, prompts[i], delimiter_id=W.DELIMITER_ID, keyword_ids=W.KEYWORD_IDS, n1=4,
                                    max_new_tokens=budgets[i], force=forces[i])
        _assert_routing_equal(want, got[i])
        assert len(got[i].tokens) == budgets[i]
        n_hand += len(want.handoffs)
    assert n_hand >= 6
    gs.close()
    gl.close()


def test_batched_generation_in_rounds(B, oracle):
    """Enough sequence slots and KV pages for all sequences: they advance together, one batched decode pass per
    model and round plus a multi-row pass per prompt / catch-up.  Routing per sequence equals the oracle's run of
    that sequence alone, and so does the greedy choice wherever the oracle's margin allows a comparison."""
    S, L = shape_dict(W.TINY_S), shape_dict(W.TINY_L)
    n = 7
    prompts, budgets, forces = W.batch_inputs(17, n, 1024, prompt_range=(5, 70), budget_range=(20, 120), mean_interval=6,
                                              keyword_rate=0.6)
    forces = [W.full_forcing(700 + i, len(f), 1024, mean_interval=6, keyword_rate=0.6) for i, f in enumerate(forces)]
    budgets[2] = 0                      # a sequence with nothing to generate
    gs = B.Model(S, seed=0, tag=0, max_seqs=n, max_tokens=n * 256)
    gl = B.Model(L, seed=0, tag=1, max_seqs=n, max_tokens=n * 256)
    got = B.st_generate_spec_batch(gs, gl, prompts, delimiter_id=W.DELIMITER_ID, keyword_ids=W.KEYWORD_IDS, n1=4,
                                   max_new_tokens=budgets, forces=forces)
    assert len({r.seconds for r in got}) == 1, "the sequences did not run as one batch"
    os_, ol = oracle.Model(oracle.Config(**S), 0, 0), oracle.Model(oracle.Config(**L), 0, 1)
    n_hand = n_cmp = 0
    for i in range(n):
        want = oracle.generate_spec(os_, ol, prompts[i], delimiter_id=W.DELIMITER_ID, keyword_ids=W.KEYWORD_IDS, n1=4,
                                    max_new_tokens=budgets[i], force=forces[i])
        _assert_routing_equal(want, got[i])
        assert len(got[i].tokens) == budgets[i]
        n_hand += len(want.handoffs)
        for t in range(len(want.emission_tokens)):
            if want.emission_margin[t] >= MARGIN:
                assert got[i].emission_argmax[t] == want.emission_argmax[t], (i, t)
                n_cmp += 1
    assert n_hand >= 6 and n_cmp >= 100
    # the models are reusable, and a second call gives the same result
    again = B.st_generate_spec_batch(gs, gl, prompts, delimiter_id=W.DELIMITER_ID, keyword_ids=W.KEYWORD_IDS, n1=4,
                                     max_new_tokens=budgets, forces=forces)
    for a, b in zip(got, again):
        assert a.tokens.tolist() == b.tokens.tolist() and a.emission_argmax.tolist() == b.emission_argmax.tolist()
    gs.close()
    gl.close()


def test_every_delimiter_variant_on_device(B, oracle):
    """The variant for a speculative model without reflective cues: the target opens the answer and takes over
    after every delimiter the small model writes.  Routing bit-exact against the oracle (hand-traced stream and a
    longer forced run), greedy choices wherever the margin allows, alone and through the batched rounds."""
    S, L = shape_dict(W.TINY_S), shape_dict(W.TINY_L)
    os_, ol = oracle.Model(oracle.Config(**S), 0, 0), oracle.Model(oracle.Config(**L), 0, 1)
    gs = B.Model(S, seed=0, tag=0, max_seqs=3, max_tokens=1024)
    gl = B.Model(L, seed=0, tag=1, max_seqs=3, max_tokens=1024)
    kw = dict(delimiter_id=W.DELIMITER_ID, keyword_ids=W.KEYWORD_IDS, takeover_every_delimiter=True)
    hand = [5, 6, 7, 10, 20, 21, 22, 8, 10, 30, 31, 32, 9]
    got = B.st_generate_spec(gs, gl, [1, 2, 3], n1=3, target_first_n=2, max_new_tokens=12, force=hand, **kw)
    assert got.tokens.tolist() == [5, 6, 7, 10, 20, 21, 22, 8, 10, 30, 31, 32]
    assert got.source.tolist() == [1, 1, 0, 0, 1, 1, 1, 0, 0, 1, 1, 1]
    assert got.handoffs == [(7, 3, 3), (12, 8, 3)]
    prompts = [W.prompt_ids(300 + i, 20 + 9 * i, 1024) for i in range(3)]
    forces = [W.full_forcing(310 + i, 300, 1024, mean_interval=7, keyword_rate=0.3) for i in range(3)]
    wants = [oracle.generate_spec(os_, ol, prompts[i], n1=5, target_first_n=10, max_new_tokens=100, force=forces[i], **kw)
             for i in range(3)]
    alone = B.st_generate_spec(gs, gl, prompts[0], n1=5, target_first_n=10, max_new_tokens=100, force=forces[0], **kw)
    batch = B.st_generate_spec_batch(gs, gl, prompts, n1=5, target_first_n=10, max_new_tokens=100, forces=forces, **kw)
    for want, got in [(wants[0], alone)] + list(zip(wants, batch)):
        _assert_routing_equal(want, got)
        assert len(want.handoffs) >= 4 and want.source[:10].tolist() == [1] * 10
        for t in range(len(want.emission_tokens)):
            if want.emission_margin[t] >= MARGIN:
                assert got.emission_argmax[t] == want.emission_argmax[t]
    gs.close()
    gl.close()


def test_batched_generation_fallbacks_and_edges(B, oracle):
    """Calls that do not qualify for the rounds (too few sequence slots or KV pages) run the sequences one by one with
    the same results; an empty batch and a single sequence are fine; a prompt longer than a pass takes its own chunks."""
    S, L = shape_dict(W.TINY_S), shape_dict(W.TINY_L)
    kw = dict(delimiter_id=W.DELIMITER_ID, keyword_ids=W.KEYWORD_IDS, n1=4)
    prompts = [W.prompt_ids(40 + i, n, 1024) for i, n in enumerate([300, 7, 33])]       # 300 > 256 rows of a pass
    forces = [W.full_forcing(50 + i, 120, 1024, mean_interval=6, keyword_rate=0.6) for i in range(3)]
    os_, ol = oracle.Model(oracle.Config(**S), 0, 0), oracle.Model(oracle.Config(**L), 0, 1)
    wants = [oracle.generate_spec(os_, ol, prompts[i], max_new_tokens=50, force=forces[i], **kw) for i in range(3)]
    roomy = (B.Model(S, seed=0, tag=0, max_seqs=3, max_tokens=2048), B.Model(L, seed=0, tag=1, max_seqs=3, max_tokens=2048))
    one_slot = (B.Model(S, seed=0, tag=0, max_seqs=1, max_tokens=2048), B.Model(L, seed=0, tag=1, max_seqs=1, max_tokens=2048))
    few_pages = (B.Model(S, seed=0, tag=0, max_seqs=3, max_tokens=512), B.Model(L, seed=0, tag=1, max_seqs=3, max_tokens=512))
    for gs, gl in (roomy, one_slot, few_pages):
        got = B.st_generate_spec_batch(gs, gl, prompts, max_new_tokens=50, forces=forces, **kw)
        for want, g in zip(wants, got):
            _assert_routing_equal(want, g)
        assert B.st_generate_spec_batch(gs, gl, [], max_new_tokens=5, **kw) == []
        single = B.st_generate_spec_batch(gs, gl, prompts[1:2], max_new_tokens=50, forces=forces[1:2], **kw)
        _assert_routing_equal(wants[1], single[0])
        # every slot is free again
        for m in (gs, gl):
            slots = [m.st_seq_alloc() for _ in range(1)]
            m.st_seq_free(slots[0])
    assert len({r.seconds for r in B.st_generate_spec_batch(*roomy, prompts, max_new_tokens=50, forces=forces, **kw)}) == 1
    for gs, gl in (roomy, one_slot, few_pages):
        gs.close()
        gl.close()


@pytest.mark.parametrize("keep", [False, True])
def test_three_takeovers_on_device(B, oracle, keep):
    """Takeovers (1)-(3) of the paper's Section 3 in token-id form (reflection / affirmation, verification by either
    model, excessive reflection with the inserted auxiliary sentence): the hand-traced stream, and a longer forced
    run against the oracle -- routing, handoff kinds and inserted tokens bit-exact, alone and in batched rounds."""
    S, L = shape_dict(W.TINY_S), shape_dict(W.TINY_L)
    os_, ol = oracle.Model(oracle.Config(**S), 0, 0), oracle.Model(oracle.Config(**L), 0, 1)
    gs = B.Model(S, seed=0, tag=0, max_seqs=3, max_tokens=1536)
    gl = B.Model(L, seed=0, tag=1, max_seqs=3, max_tokens=1536)
    rules = dict(delimiter_id=10, keyword_ids=[11, 12, 13], affirmation_ids=[14], verification_ids=[13, 15], n1=2, n2=3, n3=2,
                 neg_threshold=1, aux_ids=[40, 41])
    if not keep:
        hand = [10, 14, 20, 10, 11, 21, 10, 13, 10, 15, 22, 10, 15, 23, 24, 25, 26]
        got = B.st_generate_spec(gs, gl, [1, 2, 3], max_new_tokens=15, force=hand, **rules)
        assert got.tokens.tolist() == [10, 20, 10, 21, 10, 40, 41, 10, 15, 22, 10, 23, 24, 25, 26]
        assert got.source.tolist() == [0, 1, 1, 1, 1, 2, 2, 1, 1, 1, 1, 1, 1, 1, 0]
        assert got.handoffs == [(4, 1, 4), (6, 4, 1), (10, 7, 3), (11, 9, 0), (14, 12, 1)]
        assert got.handoff_kinds == [1, 1, 3, 2, 2]
    rules.update(n1=4, n2=9, n3=6, neg_threshold=2, aux_ids=[40, 41, 42], keep_probe=keep)
    prompts = [W.prompt_ids(500 + i, 12 + 20 * i, 1024) for i in range(3)]
    # forced streams over a small alphabet so that every class of cue follows delimiters often
    rng = np.random.default_rng(9)
    forces = [rng.choice([10, 10, 11, 13, 14, 15, 30, 31, 32, 33], size=400).astype(np.int32) for _ in range(3)]
    wants = [oracle.generate_spec(os_, ol, prompts[i], max_new_tokens=160, force=forces[i], **rules) for i in range(3)]
    assert {1, 2, 3} <= set(k for w in wants for k in w.handoff_kinds)
    alone = B.st_generate_spec(gs, gl, prompts[0], max_new_tokens=160, force=forces[0], **rules)
    batch = B.st_generate_spec_batch(gs, gl, prompts, max_new_tokens=160, forces=forces, **rules)
    for want, got in [(wants[0], alone)] + list(zip(wants, batch)):
        assert want.rc == 0
        _assert_routing_equal(want, got)
        assert got.handoff_kinds == want.handoff_kinds
        for t in range(len(want.emission_tokens)):
            if want.emission_margin[t] >= MARGIN:
                assert got.emission_argmax[t] == want.emission_argmax[t]
    gs.close()
    gl.close()


@pytest.mark.parametrize("keep", [False, True])
def test_sentence_probe_on_device(B, oracle, keep):
    """The n1-token probe sentence (paper Section 3 (1)): classified by cue counts, replaced as a whole by the target's
    segment (or kept).  The hand-traced stream, then a longer forced run with all three takeovers against the oracle:
    routing, rolled-back cache lengths, handoff kinds and greedy choices, alone and in batched rounds."""
    S, L = shape_dict(W.TINY_S), shape_dict(W.TINY_L)
    os_, ol = oracle.Model(oracle.Config(**S), 0, 0), oracle.Model(oracle.Config(**L), 0, 1)
    gs = B.Model(S, seed=0, tag=0, max_seqs=3, max_tokens=2048)
    gl = B.Model(L, seed=0, tag=1, max_seqs=3, max_tokens=2048)
    rules = dict(delimiter_id=10, keyword_ids=[11, 12], affirmation_ids=[14], verification_ids=[15], n1=3, n2=4, probe_len=3)
    if not keep:
        hand = [10, 30, 11, 14, 20, 21, 10, 14, 31, 14, 22, 23, 10, 32, 10, 33, 15, 10, 15, 34]
        got = B.st_generate_spec(gs, gl, [1, 2, 3], max_new_tokens=14, force=hand, **rules)
        assert got.tokens.tolist() == [10, 20, 21, 10, 22, 23, 10, 32, 10, 33, 15, 10, 15, 34]
        assert got.source.tolist() == [0, 1, 1, 1, 1, 1, 1, 0, 0, 0, 0, 0, 0, 0]
        assert got.handoffs == [(4, 3, 4), (7, 9, 1)] and got.handoff_kinds == [1, 1]
        assert (got.kv_len_small, got.kv_len_large) == (16, 9)
    rules.update(neg_threshold=3, n3=5, aux_ids=[40, 41], keep_probe=keep)
    rng = np.random.default_rng(4)
    forces = [rng.choice([10, 10, 11, 12, 14, 15, 30, 31, 32, 33, 34, 35], size=900).astype(np.int32) for _ in range(3)]
    prompts = [W.prompt_ids(600 + i, 9 + 30 * i, 1024) for i in range(3)]
    wants = [oracle.generate_spec(os_, ol, prompts[i], max_new_tokens=180, force=forces[i], **rules) for i in range(3)]
    assert {1, 2, 3} <= set(k for w in wants for k in w.handoff_kinds)
    alone = B.st_generate_spec(gs, gl, prompts[1], max_new_tokens=180, force=forces[1], **rules)
    batch = B.st_generate_spec_batch(gs, gl, prompts, max_new_tokens=180, forces=forces, **rules)
    for want, got in [(wants[1], alone)] + list(zip(wants, batch)):
        assert want.rc == 0
        _assert_routing_equal(want, got)
        assert got.handoff_kinds == want.handoff_kinds
        for t in range(len(want.emission_tokens)):
            if want.emission_margin[t] >= MARGIN:
                assert got.emission_argmax[t] == want.emission_argmax[t]
    gs.close()
    gl.close()


def test_hand_traced_rule_cases_on_device(B):
    """The hand-traced streams of tests/golden (cue precedence inside a probe sentence, the reflection counter
    crossing its threshold and restarting, probe sentences cut by end-of-sequence or the budget in both probe
    readings, a delimiter inside a probe, verification cues in the target's own sentences): the device's
    routing must reproduce every one of them bit for bit, alone and in batched rounds.  No oracle is involved:
    the expected values were traced by hand from the paper's rules."""
    from test_oracle_spec import RULE_TRACES, assert_matches_trace, load_rule_trace
    S, L = shape_dict(W.TINY_S), shape_dict(W.TINY_L)
    gs = B.Model(S, seed=0, tag=0, max_seqs=2, max_tokens=512)
    gl = B.Model(L, seed=0, tag=1, max_seqs=2, max_tokens=512)
    for name in RULE_TRACES:
        T, params = load_rule_trace(name)
        got = B.st_generate_spec(gs, gl, T["prompt"], max_new_tokens=T["max_new"], force=T["force"], **params)
        assert_matches_trace(got, T)
        twice = B.st_generate_spec_batch(gs, gl, [T["prompt"], T["prompt"]], max_new_tokens=T["max_new"],
                                         forces=[T["force"], T["force"]], **params)
        for r in twice:
            assert_matches_trace(r, T)
        if "budget" in T:
            cut = B.st_generate_spec(gs, gl, T["prompt"], max_new_tokens=T["budget"], force=T["force"], **dict(params, eos_id=-1))
            assert cut.tokens.tolist() == T["budget_tokens"] and len(cut.emission_tokens) == T["budget_steps"]
            assert cut.handoffs == T["handoffs"]
    gs.close()
    gl.close()


def test_phase_times_and_pass_counts(B):
    """The per-kind device times of st_spec_result (the split of the paper's Table "comparison of time"): the pass
    counts must equal what the emission log says (one token ingested = decode, a model's first tokens = prompt
    prefill, anything else = catch-up) and the three times must add up to the generation's device time."""
    S, L = shape_dict(W.TINY_S), shape_dict(W.TINY_L)
    gs = B.Model(S, seed=0, tag=0, max_tokens=1024)
    gl = B.Model(L, seed=0, tag=1, max_tokens=1024)
    prompt = W.prompt_ids(100, 300, 1024)          # longer than one 256-row pass: the prompt prefill is chunked
    force = W.full_forcing(101, 1200, 1024, mean_interval=8, keyword_rate=0.5)
    r = B.st_generate_spec(gs, gl, prompt, delimiter_id=W.DELIMITER_ID, keyword_ids=W.KEYWORD_IDS, n1=5, max_new_tokens=400, force=force)
    fed, src = r.emission_fed, r.emission_source
    pt = r.phase_times
    first = {int(m): int(np.argmax(src == m)) for m in (0, 1) if (src == m).any()}
    n_prompt = sum(1 for m, t in first.items() if fed[t] > 1)
    assert pt["decode"][1] == int((fed == 1).sum())
    assert pt["prompt_prefill"][1] == n_prompt == 2
    assert pt["catchup"][1] == int((fed > 1).sum()) - n_prompt and pt["catchup"][1] >= 5
    total = sum(v[0] for v in pt.values())
    assert all(v[0] > 0 for v in pt.values())
    assert abs(total - r.seconds) <= 0.1 * r.seconds + 2e-4, (total, r.seconds)
    gs.close()
    gl.close()


@pytest.mark.parametrize("temperature", [0.7, 1.5])
def test_temperature_sampling_on_device(B, oracle, temperature):
    """Tokens drawn by the Gumbel-max rule (temperature sampling with a counter-based generator): under teacher
    forcing with the oracle's stream, the token the device draws at every step equals the oracle's wherever the
    oracle's decision is clear (gap of the two largest perturbed logits at least the tolerance, scaled by 1 / T);
    handoffs triggered by drawn tokens follow; the same seed reproduces the run and another seed changes it."""
    S, L = shape_dict(W.TINY_S), shape_dict(W.TINY_L)
    os_, ol = oracle.Model(oracle.Config(**S), 0, 0), oracle.Model(oracle.Config(**L), 0, 1)
    gs = B.Model(S, seed=0, tag=0, max_tokens=512)
    gl = B.Model(L, seed=0, tag=1, max_tokens=512)
    prompt = W.prompt_ids(100, 32, 1024)
    sched = W.forcing_schedule(101, 400, mean_interval=8, keyword_rate=0.5)   # delimiters and keywords forced, the rest drawn
    kw = dict(delimiter_id=W.DELIMITER_ID, keyword_ids=W.KEYWORD_IDS, n1=4, max_new_tokens=120, temperature=temperature, sample_seed=77)
    want = oracle.generate_spec(os_, ol, prompt, force=sched, **kw)
    assert len(want.handoffs) >= 3
    forced = B.st_generate_spec(gs, gl, prompt, force=want.emission_tokens, **kw)
    _assert_routing_equal(want, forced)
    clear = want.emission_margin >= MARGIN * max(1.0, 1.0 / temperature)
    assert clear.sum() >= 60
    assert forced.emission_argmax[clear].tolist() == want.emission_argmax[clear].tolist()
    # drawn tokens differ from the greedy ones
    greedy = oracle.generate_spec(os_, ol, prompt, force=sched, **dict(kw, temperature=0.0))
    assert want.tokens.tolist() != greedy.tokens.tolist()
    # free-running: identical up to the first unclear decision; reproducible; seed-dependent
    free = B.st_generate_spec(gs, gl, prompt, force=sched, **kw)
    again = B.st_generate_spec(gs, gl, prompt, force=sched, **kw)
    other = B.st_generate_spec(gs, gl, prompt, force=sched, **dict(kw, sample_seed=78))
    assert free.tokens.tolist() == again.tokens.tolist() != other.tokens.tolist()
    for t in range(min(len(free.emission_tokens), len(want.emission_tokens))):
        if free.emission_tokens[t] != want.emission_tokens[t]:
            assert not clear[t], f"step {t}: drawn tokens differ at a clear margin"
            break
    gs.close()
    gl.close()


@pytest.mark.parametrize("top_p", [0.5, 0.9])
def test_top_p_sampling_on_device(B, oracle, top_p):
    """Top-p (nucleus) sampling: under teacher forcing with the oracle's stream, the token the device draws equals the
    oracle's at every step where the oracle's decision is clear -- the gap of the two largest perturbed logits at least
    the tolerance, and the same token wins for every nucleus between those of top_p - 0.03 and top_p + 0.03 (the sets
    are nested, so one winner at both ends is the winner of every set in between; the device sums the probability mass
    in single precision from its own logits, which moves the cut by a few boundary ids at most).  Covers the decode kernel's in-kernel cut and the cut that precedes
    the sampling kernel of multi-row passes (the first token after the prompt, every token after a catch-up)."""
    S, L = shape_dict(W.TINY_S), shape_dict(W.TINY_L)
    os_, ol = oracle.Model(oracle.Config(**S), 0, 0), oracle.Model(oracle.Config(**L), 0, 1)
    gs = B.Model(S, seed=0, tag=0, max_tokens=512)
    gl = B.Model(L, seed=0, tag=1, max_tokens=512)
    prompt = W.prompt_ids(100, 32, 1024)
    sched = W.forcing_schedule(101, 400, mean_interval=8, keyword_rate=0.5)
    T = 1.0
    kw = dict(delimiter_id=W.DELIMITER_ID, keyword_ids=W.KEYWORD_IDS, n1=4, max_new_tokens=120, temperature=T, sample_seed=77,
              top_p=top_p)
    want = oracle.generate_spec(os_, ol, prompt, force=sched, trace_n_steps=400, **kw)
    n = len(want.emission_tokens)
    ends = [[oracle.sample_top_p(want.logits_trace[t], T, q, 77, t)[:2] for q in (top_p - 0.03, top_p + 0.03)] for t in range(n)]
    robust = np.array([lo[0] == hi[0] and min(lo[1], hi[1]) >= MARGIN for lo, hi in ends])
    forced = B.st_generate_spec(gs, gl, prompt, force=want.emission_tokens, **kw)
    _assert_routing_equal(want, forced)
    clear = (want.emission_margin >= MARGIN) & robust
    assert clear.sum() >= 50
    assert forced.emission_argmax[clear].tolist() == want.emission_argmax[clear].tolist()
    # the restriction matters: the unrestricted draws differ somewhere, and every drawn token lies in the oracle's nucleus
    free = oracle.generate_spec(os_, ol, prompt, force=sched, **dict(kw, top_p=0.0))
    assert free.emission_argmax.tolist() != want.emission_argmax.tolist()
    for t in np.flatnonzero(clear):
        thr = oracle.nucleus_threshold(want.logits_trace[t], T, top_p)[0]
        assert want.logits_trace[t][forced.emission_argmax[t]] >= thr
    # top_p = 1 is plain temperature sampling
    a = B.st_generate_spec(gs, gl, prompt, force=sched, **dict(kw, top_p=1.0))
    b = B.st_generate_spec(gs, gl, prompt, force=sched, **dict(kw, top_p=0.0))
    assert a.tokens.tolist() == b.tokens.tolist()
    gs.close()
    gl.close()


def test_top_p_large_vocabulary(B, oracle):
    """The nucleus cut over a vocabulary of 151 936 ids (two layers at the 1.5B's widths): all three histogram levels
    of the device's threshold search are exercised with ~10^5 ids inside the nucleus."""
    import dataclasses
    shape = shape_dict(dataclasses.replace(W.QWEN_1P5B, n_layers=2))
    om = oracle.Model(oracle.Config(**shape), 0, 0)
    gm = B.Model(shape, seed=0, tag=0, max_tokens=256)
    prompt = W.prompt_ids(5, 12, shape["vocab"])
    T, top_p = 0.8, 0.7
    kw = dict(delimiter_id=W.DELIMITER_ID, keyword_ids=[], n1=4, max_new_tokens=10, temperature=T, sample_seed=11, top_p=top_p)
    want = oracle.generate_spec(om, None, prompt, trace_n_steps=16, **kw)
    n = len(want.emission_tokens)
    forced = B.st_generate_spec(gm, None, prompt, force=want.emission_tokens, **kw)
    ends = [[oracle.sample_top_p(want.logits_trace[t], T, q, 11, t)[:2] for q in (top_p - 0.03, top_p + 0.03)] for t in range(n)]
    clear = np.array([lo[0] == hi[0] and min(lo[1], hi[1]) >= MARGIN for lo, hi in ends]) & (want.emission_margin >= MARGIN)
    assert clear.sum() >= 5
    assert forced.emission_argmax[clear].tolist() == want.emission_argmax[clear].tolist()
    # the cut removes a real share of the vocabulary and the unrestricted draw differs somewhere
    inside = [(want.logits_trace[t] >= oracle.nucleus_threshold(want.logits_trace[t], T, top_p)[0]).sum() for t in range(n)]
    assert 1000 < min(inside) and max(inside) < shape["vocab"] - 1000
    gm.close()
