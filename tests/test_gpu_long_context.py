"""GPU parity at the contexts the benchmark runs: logits against the CPU oracle where the decode kernel's
attention unit streams its keys through the staging area in several chunks, where multi-row passes attend
over thousands of cached keys, where a batched step holds 64 ragged sequences, and where multi-row passes run
deeper than two layers.

Cost control on the oracle side: its attention is quadratic in the context and its projections cost
2 * parameters per row, so the long contexts use either narrowed widths (true head layout, two layers) or the
true widths with one layer, together with KV.forward_last (which leaves out rows nothing reads and is pinned to
the full pass on the CPU).  Every case asserts from the library's own geometry report that it takes the
multi-chunk path it is meant to cover."""
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
    build.build()
    binding.lib()
    return binding


def _prefill_both(gm, slot, okv, tokens, logits):
    """Ingest `tokens` on both sides (the GPU in passes of at most 256 rows); returns (got, want) of the last row."""
    n = len(tokens)
    for i in range(0, n, 256):
        last = i + 256 >= n
        gm.st_prefill(slot, tokens[i:i + 256], logits if last else None)
    want = okv.forward_last(tokens)
    torch.cuda.synchronize()
    return logits.cpu().numpy(), want


def _long_context(B, oracle, shape, ctx, *, rows_after=(), n_decode=3, page_size=64, min_chunks=3, tag=3, seed=0,
                  want_empty_own_chunk=False, tok_seed=5):
    rng = np.random.default_rng(tok_seed)
    total = ctx + sum(rows_after) + n_decode
    tokens = rng.integers(0, shape["vocab"], size=total).astype(np.int32)
    om = oracle.Model(oracle.Config(**shape), seed, tag)
    okv = oracle.KV(om, total + 1)
    gm = B.Model(shape, seed=seed, tag=tag, max_seqs=1, max_tokens=total + 64, page_size=page_size)
    slot = gm.st_seq_alloc()
    logits = torch.empty(shape["vocab"], dtype=torch.float32, device="cuda")
    worst = [0.0, 1.0]

    def check(got, want, what):
        e, cs = assert_logits_close(got, want, what)
        worst[0], worst[1] = max(worst[0], e), min(worst[1], cs)

    got, want = _prefill_both(gm, slot, okv, tokens[:ctx], logits)
    check(got, want, f"last row of the {ctx}-token prompt")
    i = ctx
    for r in rows_after:   # catch-up sized passes over the long context (multi-row attention with key splits)
        got, want = _prefill_both(gm, slot, okv, tokens[i:i + r], logits)
        check(got, want, f"{r}-row pass over {i} cached tokens")
        i += r
    tok_dev = torch.empty(1, dtype=torch.int32, device="cuda")
    amax = torch.empty(1, dtype=torch.int32, device="cuda")
    chunks_seen, empty_seen = [], False
    for _ in range(n_decode):
        geo = gm.st_decode_geometry(i)
        chunks_seen.append(geo["max_chunks"])
        empty_seen = empty_seen or geo["own_chunk_empty"]
        want = okv.forward(tokens[i:i + 1])
        tok_dev.copy_(torch.from_numpy(tokens[i:i + 1]))
        gm.st_decode_step([slot], tok_dev, logits, amax)
        torch.cuda.synchronize()
        got = logits.cpu().numpy()
        check(got, want, f"decode at {i} ({geo})")
        gi, margin = oracle.argmax(want)
        if margin >= MARGIN:
            assert int(amax.item()) == gi
        assert int(amax.item()) == int(np.argmax(got))
        i += 1
        assert gm.st_kv_len(slot) == i
    assert gm.st_last_device_status() == 0
    # the case is only worth its time if the decode steps really streamed several staging chunks
    assert min(chunks_seen) >= min_chunks, (chunks_seen, gm.st_decode_geometry(ctx))
    if want_empty_own_chunk:
        assert empty_seen, "no step had its own key alone in the last chunk"
    gm.close()
    print(f"ctx {ctx}, {shape['n_q_heads']}/{shape['n_kv_heads']} heads x {shape['n_layers']} layers: chunks {chunks_seen}, "
          f"worst max-abs {worst[0]:.4f}, worst cosine {worst[1]:.7f}")


@pytest.mark.parametrize("shape,tag", [(W.TINY_S, 0), (W.TINY_L, 1)])
@pytest.mark.parametrize("page_size", [16, 64])
@pytest.mark.parametrize("cap", [32, 48])
def test_small_staging_area_streams_chunks(B, oracle, monkeypatch, shape, tag, page_size, cap):
    """With the staging area clamped to 32 / 48 keys the tiny models stream units of ~64 keys in 16- / 24-key
    chunks (so 3 to 5 chunks, refills included); 24 consecutive steps include one whose own key is alone in the
    last chunk (an empty transfer)."""
    monkeypatch.setenv("ST_MEGA_KV_CAP", str(cap))
    _long_context(B, oracle, shape_dict(shape), 690, n_decode=24, page_size=page_size, min_chunks=3, tag=tag,
                  want_empty_own_chunk=(cap == 32))


def _real_staging_cap(B, shape):
    """Staging capacity (keys) of the decode kernel for the full-width model of `shape` (one layer is enough)."""
    gm = B.Model(shape_dict(shape, n_layers=1, vocab=1024), seed=0, tag=9, max_seqs=1, max_tokens=256)
    cap = gm.st_decode_geometry(0)["kv_cap"]
    gm.close()
    return cap


@pytest.mark.parametrize("shape,ctx,min_chunks", [(W.QWEN_32B, 3000, 3), (W.QWEN_7B, 6200, 2)])
def test_head_layouts_two_layers_long_context(B, oracle, monkeypatch, shape, ctx, min_chunks):
    """The large models' head layouts (40 q / 8 kv and 28 q / 4 kv heads of 128) two layers deep with hidden, FFN
    and vocabulary narrowed, the staging capacity set to the full-width model's: decode steps plus a 20-row and a
    130-row catch-up over the long context."""
    cap = _real_staging_cap(B, shape)
    monkeypatch.setenv("ST_MEGA_KV_CAP", str(cap))
    narrowed = shape_dict(shape, n_layers=2, hidden=1024, ffn=2048, vocab=4096)
    _long_context(B, oracle, narrowed, ctx, rows_after=(20, 130), n_decode=3, min_chunks=min_chunks)


@pytest.mark.parametrize("shape,ctx,page_size,min_chunks", [(W.QWEN_32B, 3000, 64, 3), (W.QWEN_32B, 12300, 16, 8),
                                                             (W.QWEN_7B, 6200, 64, 2)])
def test_true_width_one_layer_long_context(B, oracle, shape, ctx, page_size, min_chunks):
    """The true hidden / FFN widths (so the decode kernel has exactly the shared-memory layout, split count and
    staging capacity of the full model), one layer, at the contexts of the benchmark's middle and end: decode
    steps and catch-up passes of 20 and 130 rows."""
    _long_context(B, oracle, shape_dict(shape, n_layers=1, vocab=4096), ctx, rows_after=(20, 130), n_decode=3,
                  page_size=page_size, min_chunks=min_chunks)


def test_batched_step_64_ragged_sequences_true_width(B, oracle):
    """st_decode_step with 64 sequences of ragged cached lengths from 1 to 4000 on the 32B's true widths (one
    layer, so that the oracle's prefill stays linear in the cached rows): every row's logits against the oracle
    run on that sequence alone."""
    shape = shape_dict(W.QWEN_32B, n_layers=1, vocab=4096)
    rng = np.random.default_rng(21)
    n, n_steps = 64, 2
    # a few long sequences among many short ones: the oracle's cost grows with the total number of cached rows
    lengths = [4000, 3071, 2049, 1000, 517, 1] + [int(x) for x in rng.integers(2, 200, size=n - 6)]
    om = oracle.Model(oracle.Config(**shape), 0, 2)
    gm = B.Model(shape, seed=0, tag=2, max_seqs=n, max_tokens=sum(lengths) + n * (n_steps + 64))
    okvs, slots, toks = [], [], []
    for ln in lengths:
        t = rng.integers(0, shape["vocab"], size=ln + n_steps).astype(np.int32)
        okv = oracle.KV(om, ln + n_steps + 1)
        okv.forward_last(t[:ln])
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
    assert gm.st_last_device_status() == 0
    gm.close()
    print(f"64 ragged sequences: worst max-abs {worst:.4f}")


def test_multi_row_passes_eight_layers_deep(B, oracle):
    """A 256-row prompt pass and a 130-row catch-up over it at the 32B's widths, eight layers deep: the error of
    the split-plane tensor-core projections must stay inside the tolerance as depth grows."""
    shape = shape_dict(W.QWEN_32B, n_layers=8, vocab=4096)
    rng = np.random.default_rng(8)
    tokens = rng.integers(0, shape["vocab"], size=256 + 130 + 2).astype(np.int32)
    om = oracle.Model(oracle.Config(**shape), 0, 3)
    okv = oracle.KV(om, len(tokens) + 1)
    gm = B.Model(shape, seed=0, tag=3, max_seqs=1, max_tokens=len(tokens) + 64)
    slot = gm.st_seq_alloc()
    logits = torch.empty(shape["vocab"], dtype=torch.float32, device="cuda")
    worst = 0.0
    i = 0
    for rows in (256, 130):
        want = okv.forward(tokens[i:i + rows])
        gm.st_prefill(slot, tokens[i:i + rows], logits)
        torch.cuda.synchronize()
        e, cs = assert_logits_close(logits.cpu().numpy(), want, f"{rows}-row pass at {i}, 8 layers")
        worst = max(worst, e)
        i += rows
    tok_dev = torch.empty(1, dtype=torch.int32, device="cuda")
    for _ in range(2):
        want = okv.forward(tokens[i:i + 1])
        tok_dev.copy_(torch.from_numpy(tokens[i:i + 1]))
        gm.st_decode_step([slot], tok_dev, logits, None)
        torch.cuda.synchronize()
        e, cs = assert_logits_close(logits.cpu().numpy(), want, f"decode at {i} on top of the multi-row passes")
        worst = max(worst, e)
        i += 1
    assert gm.st_last_device_status() == 0
    gm.close()
    print(f"8 layers: worst max-abs {worst:.4f}")


def test_kv_truncate_then_refeed(B, oracle):
    """st_kv_truncate drops cached positions; feeding the dropped tokens again (as one multi-row pass, then
    again as single steps after a second truncation) reproduces the oracle's logits after the same truncation."""
    shape = shape_dict(W.TINY_L)
    rng = np.random.default_rng(13)
    tokens = rng.integers(0, shape["vocab"], size=150).astype(np.int32)
    other = rng.integers(0, shape["vocab"], size=40).astype(np.int32)
    om = oracle.Model(oracle.Config(**shape), 0, 1)
    okv = oracle.KV(om, 256)
    gm = B.Model(shape, seed=0, tag=1, max_seqs=1, max_tokens=512, page_size=16)
    slot = gm.st_seq_alloc()
    logits = torch.empty(shape["vocab"], dtype=torch.float32, device="cuda")
    gm.st_prefill(slot, tokens, logits)
    okv.forward(tokens)
    # roll back 40 positions and write different tokens there
    gm.st_kv_truncate(slot, 110)
    okv.truncate(110)
    assert gm.st_kv_len(slot) == 110
    want = okv.forward(other)
    gm.st_prefill(slot, other, logits)
    torch.cuda.synchronize()
    assert_logits_close(logits.cpu().numpy(), want, "multi-row re-feed after truncation")
    assert gm.st_kv_len(slot) == 150
    # truncating to a larger length changes nothing
    gm.st_kv_truncate(slot, 400)
    assert gm.st_kv_len(slot) == 150
    # roll back across a page boundary and re-feed token by token through the decode kernel
    gm.st_kv_truncate(slot, 95)
    okv.truncate(95)
    tok_dev = torch.empty(1, dtype=torch.int32, device="cuda")
    for j in range(6):
        want = okv.forward(tokens[95 + j:96 + j])
        tok_dev.copy_(torch.from_numpy(tokens[95 + j:96 + j]))
        gm.st_decode_step([slot], tok_dev, logits, None)
        torch.cuda.synchronize()
        assert_logits_close(logits.cpu().numpy(), want, f"decode re-feed {j} after truncation")
    assert gm.st_kv_len(slot) == 101
    assert gm.st_last_device_status() == 0
    gm.close()
