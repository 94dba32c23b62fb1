"""Pins for the oracle's transformer forward: a library implementation of the same architecture,
a model small enough to work by hand, and the cache invariants (CPU only)."""
import math

import numpy as np
import pytest
import torch


def _cfg(oracle, **kw):
    base = dict(n_layers=2, hidden=64, n_q_heads=4, n_kv_heads=2, head_dim=16, ffn=128, vocab=97,
                rope_theta=1e4, rms_eps=1e-6, tie_embeddings=1, qkv_bias=1)
    base.update(kw)
    return oracle.Config(**base)


def _hf_model(oracle, cfg, seed, tag, gains=None):
    from transformers import Qwen2Config, Qwen2ForCausalLM
    hc = Qwen2Config(vocab_size=cfg.vocab, hidden_size=cfg.hidden, intermediate_size=cfg.ffn,
                     num_hidden_layers=cfg.n_layers, num_attention_heads=cfg.n_q_heads,
                     num_key_value_heads=cfg.n_kv_heads, head_dim=cfg.head_dim, rope_theta=cfg.rope_theta,
                     rms_norm_eps=cfg.rms_eps, tie_word_embeddings=bool(cfg.tie_embeddings),
                     max_position_embeddings=512, attn_implementation="eager", use_sliding_window=False)
    m = Qwen2ForCausalLM(hc).double().eval()
    h, qd, kd, f = cfg.hidden, cfg.n_q_heads * cfg.head_dim, cfg.n_kv_heads * cfg.head_dim, cfg.ffn

    def T(tid, *shape):
        n = int(np.prod(shape))
        return torch.from_numpy(oracle.fill_tensor(seed, tag, tid, 0, n).astype(np.float64).reshape(shape))

    sd = {"model.embed_tokens.weight": T(0, cfg.vocab, h)}
    sd["lm_head.weight"] = sd["model.embed_tokens.weight"] if cfg.tie_embeddings else T(1, cfg.vocab, h)
    sd["model.norm.weight"] = torch.ones(h, dtype=torch.float64) if gains is None else torch.from_numpy(gains["final"])
    for l in range(cfg.n_layers):
        p, t = f"model.layers.{l}.", 16 * (l + 1)
        sd[p + "self_attn.q_proj.weight"] = T(t + 1, qd, h)
        sd[p + "self_attn.k_proj.weight"] = T(t + 2, kd, h)
        sd[p + "self_attn.v_proj.weight"] = T(t + 3, kd, h)
        sd[p + "self_attn.q_proj.bias"] = T(t + 4, qd)
        sd[p + "self_attn.k_proj.bias"] = T(t + 5, kd)
        sd[p + "self_attn.v_proj.bias"] = T(t + 6, kd)
        sd[p + "self_attn.o_proj.weight"] = T(t + 7, h, qd)
        sd[p + "mlp.gate_proj.weight"] = T(t + 9, f, h)
        sd[p + "mlp.up_proj.weight"] = T(t + 10, f, h)
        sd[p + "mlp.down_proj.weight"] = T(t + 11, h, f)
        sd[p + "input_layernorm.weight"] = torch.ones(h, dtype=torch.float64) if gains is None else torch.from_numpy(gains[(l, 0)])
        sd[p + "post_attention_layernorm.weight"] = torch.ones(h, dtype=torch.float64) if gains is None else torch.from_numpy(gains[(l, 8)])
    missing, unexpected = m.load_state_dict(sd, strict=False)
    assert not unexpected and all("rotary" in k or "lm_head" in k for k in missing), (missing, unexpected)
    return m


@pytest.mark.parametrize("tied,gqa", [(1, (4, 2)), (0, (4, 4)), (1, (6, 1))])
def test_forward_matches_library_qwen2(oracle, tied, gqa):
    """The same weights in the transformers library's Qwen2 (float64, eager attention) give the same logits.
    Pins norm placement, bias use, rotary pairing, grouped-query head mapping, SwiGLU and weight tying."""
    cfg = _cfg(oracle, tie_embeddings=tied, n_q_heads=gqa[0], n_kv_heads=gqa[1], hidden=gqa[0] * 16)
    rng = np.random.default_rng(5)
    gains = {"final": 1.0 + 0.3 * rng.standard_normal(cfg.hidden)}
    for l in range(cfg.n_layers):
        gains[(l, 0)] = 1.0 + 0.3 * rng.standard_normal(cfg.hidden)
        gains[(l, 8)] = 1.0 + 0.3 * rng.standard_normal(cfg.hidden)
    om = oracle.Model(cfg, 7, 3)
    om.set_gain(-1, 0, gains["final"])
    for l in range(cfg.n_layers):
        om.set_gain(l, 0, gains[(l, 0)])
        om.set_gain(l, 8, gains[(l, 8)])
    hf = _hf_model(oracle, cfg, 7, 3, gains)
    tokens = rng.integers(0, cfg.vocab, size=23).astype(np.int32)
    with torch.no_grad():
        want = hf(torch.from_numpy(tokens.astype(np.int64))[None]).logits[0].numpy()
    assert np.abs(want).max() > 0.05
    # the library builds its cos/sin tables in float32, hence 1e-6 rather than 1e-12; a wrong pairing,
    # sign, head mapping or norm placement moves logits by ~1e-1
    full = om.forward_full(tokens)
    assert np.allclose(full, want, atol=1e-6)
    kv = oracle.KV(om, 64)
    assert np.allclose(kv.forward(tokens, all_rows=True), want, atol=1e-6)


def test_generated_weights_equal_materialised(oracle):
    cfg = _cfg(oracle)
    tokens = np.arange(9, dtype=np.int32) * 5 % cfg.vocab
    a = oracle.Model(cfg, 11, 2, materialize=True).forward_full(tokens)
    b = oracle.Model(cfg, 11, 2, materialize=False).forward_full(tokens)
    assert np.array_equal(a, b)


def test_cached_decode_equals_full_recompute(oracle):
    cfg = _cfg(oracle)
    om = oracle.Model(cfg, 1, 0)
    rng = np.random.default_rng(9)
    tokens = rng.integers(0, cfg.vocab, size=19).astype(np.int32)
    full = om.forward_full(tokens)
    # (a) token by token
    kv = oracle.KV(om, 32)
    for i, t in enumerate(tokens):
        z = kv.forward([t])
        assert np.allclose(z, full[i], atol=1e-12)
        assert len(kv) == i + 1
    # (b) any chunking of the prefill gives the one-shot result: the catch-up invariant
    for chunks in ([19], [1, 18], [7, 1, 1, 10], [5, 5, 5, 4]):
        kv = oracle.KV(om, 32)
        rows, i = [], 0
        for c in chunks:
            rows.append(kv.forward(tokens[i:i + c], all_rows=True))
            i += c
        assert np.allclose(np.concatenate(rows), full, atol=1e-12)
    # (c) truncation then re-feeding reproduces the same logits
    kv.truncate(10)
    assert len(kv) == 10
    assert np.allclose(kv.forward(tokens[10:], all_rows=True), full[10:], atol=1e-12)
    # (d) a prefix's logits do not depend on what follows (causality)
    assert np.allclose(om.forward_full(tokens[:8]), full[:8], atol=1e-12)


def test_last_row_only_pass_equals_full_pass(oracle):
    """forward_last leaves out work nothing reads; its logits and its cache must equal forward's, for one and
    several layers, from an empty and from a filled cache, and later steps on top of either cache must agree."""
    rng = np.random.default_rng(4)
    for n_layers in (1, 2, 3):
        cfg = _cfg(oracle, n_layers=n_layers)
        om = oracle.Model(cfg, 2, 0)
        tokens = rng.integers(0, cfg.vocab, size=23).astype(np.int32)
        full = om.forward_full(tokens)
        a, b = oracle.KV(om, 32), oracle.KV(om, 32)
        for lo, hi in ((0, 9), (9, 10), (10, 21)):
            za, zb = a.forward(tokens[lo:hi]), b.forward_last(tokens[lo:hi])
            assert np.array_equal(za, zb)
            assert np.allclose(zb, full[hi - 1], atol=1e-12)
            assert len(a) == len(b) == hi
        # the caches are interchangeable afterwards
        assert np.array_equal(a.forward(tokens[21:22]), b.forward(tokens[21:22]))
        assert np.allclose(b.forward(tokens[22:23]), full[22], atol=1e-12)


def test_gqa_equals_mha_with_repeated_kv(oracle):
    cfg_g = _cfg(oracle, n_layers=1, n_q_heads=4, n_kv_heads=2)
    cfg_m = _cfg(oracle, n_layers=1, n_q_heads=4, n_kv_heads=4)
    g, m = oracle.Model(cfg_g, 4, 0), oracle.Model(cfg_m, 4, 0)
    d, h = cfg_g.head_dim, cfg_g.hidden
    t = 16
    for wsel, bsel in ((oracle.WK, oracle.BK), (oracle.WV, oracle.BV)):
        w = oracle.fill_tensor(4, 0, t + wsel, 0, 2 * d * h).reshape(2, d, h)
        b = oracle.fill_tensor(4, 0, t + bsel, 0, 2 * d).reshape(2, d)
        m.set_tensor(0, wsel, np.repeat(w, 2, axis=0))     # q heads 0,1 -> kv head 0; 2,3 -> kv head 1
        m.set_tensor(0, bsel, np.repeat(b, 2, axis=0))
    tokens = np.array([3, 50, 7, 7, 96, 1], dtype=np.int32)
    assert np.allclose(g.forward_full(tokens), m.forward_full(tokens), atol=1e-12)


def test_hand_worked_model(oracle):
    """One layer, hidden 2, one head of width 2, FFN width 1, vocab 2, untied head, no biases; two tokens.
    Every number below is worked out from the layer definitions with scalar arithmetic."""
    cfg = oracle.Config(n_layers=1, hidden=2, n_q_heads=1, n_kv_heads=1, head_dim=2, ffn=1, vocab=2,
                        rope_theta=1e4, rms_eps=0.0, tie_embeddings=0, qkv_bias=0)
    m = oracle.Model(cfg, 0, 0)
    E = np.array([[1.0, 0.0], [0.0, 2.0]])
    m.set_tensor(-1, oracle.EMBED, E)
    m.set_tensor(-1, oracle.LMHEAD, [[1.0, 0.0], [0.0, 1.0]])
    m.set_tensor(0, oracle.WQ, [[1.0, 0.0], [0.0, 1.0]])
    m.set_tensor(0, oracle.WK, [[1.0, 0.0], [0.0, 1.0]])
    m.set_tensor(0, oracle.WV, [[0.0, 1.0], [1.0, 0.0]])      # v swaps the two coordinates
    m.set_tensor(0, oracle.WO, [[0.5, 0.0], [0.0, 0.5]])
    m.set_tensor(0, oracle.WG, [[1.0, 1.0]])
    m.set_tensor(0, oracle.WU, [[1.0, -1.0]])
    m.set_tensor(0, oracle.WD, [[1.0], [2.0]])
    r2 = math.sqrt(2.0)
    # token 0 at position 0: x=(1,0); rms -> (sqrt2,0); q=k=(sqrt2,0) (no rotation at p=0); v=(0,sqrt2)
    # single key -> attn = v; x1 = x + 0.5*v = (1, sqrt2/2)
    x1 = np.array([1.0, r2 / 2])
    # ffn: xn = x1/sqrt(mean sq) with mean sq = (1+0.5)/2 = 0.75
    s = math.sqrt(0.75)
    xn = x1 / s
    gate, up = xn[0] + xn[1], xn[0] - xn[1]
    a = gate / (1.0 + math.exp(-gate)) * up
    x2 = x1 + np.array([a, 2 * a])
    logits0 = x2 / math.sqrt((x2 ** 2).mean())
    # token 1 at position 1: x=(0,2); rms -> (0,sqrt2); q=k=R_1(0,sqrt2) = (-sqrt2 sin1, sqrt2 cos1); v=(sqrt2,0)
    q1 = np.array([-r2 * math.sin(1.0), r2 * math.cos(1.0)])
    k0 = np.array([r2, 0.0])
    s0, s1 = q1 @ k0 / r2, q1 @ q1 / r2                      # scale 1/sqrt(d) = 1/sqrt2
    w0 = math.exp(s0) / (math.exp(s0) + math.exp(s1))
    attn = w0 * np.array([0.0, r2]) + (1 - w0) * np.array([r2, 0.0])
    y1 = np.array([0.0, 2.0]) + 0.5 * attn
    yn = y1 / math.sqrt((y1 ** 2).mean())
    gate, up = yn[0] + yn[1], yn[0] - yn[1]
    a = gate / (1.0 + math.exp(-gate)) * up
    y2 = y1 + np.array([a, 2 * a])
    logits1 = y2 / math.sqrt((y2 ** 2).mean())
    got = m.forward_full(np.array([0, 1], dtype=np.int32))
    assert np.allclose(got[0], logits0, atol=1e-14)
    assert np.allclose(got[1], logits1, atol=1e-14)
    kv = oracle.KV(m, 4)
    assert np.allclose(kv.forward([0, 1], all_rows=True), got, atol=1e-14)
