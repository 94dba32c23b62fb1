"""Pins for the oracle's layer primitives: closed forms, invariants and library routines (CPU only)."""
import math

import numpy as np
import torch
import torch.nn.functional as F


def test_rmsnorm_properties_and_library(oracle):
    rng = np.random.default_rng(1)
    x = rng.standard_normal(96)
    g = rng.standard_normal(96)
    y = oracle.rmsnorm(x, None, 0.0)
    assert abs(np.sqrt((y ** 2).mean()) - 1.0) < 1e-12              # unit RMS for unit gains
    assert np.allclose(oracle.rmsnorm(-3.5 * x, None, 0.0), -y, atol=1e-12)   # scale invariance up to sign
    want = F.rms_norm(torch.from_numpy(x), (96,), torch.from_numpy(g), eps=1e-6).numpy()
    assert np.allclose(oracle.rmsnorm(x, g, 1e-6), want, atol=1e-13)
    # eps matters when x is tiny: x/sqrt(eps)
    tiny = np.full(8, 1e-9)
    assert np.allclose(oracle.rmsnorm(tiny, None, 1e-6), tiny / math.sqrt(1e-18 + 1e-6), rtol=1e-12)


def test_silu(oracle):
    assert oracle.silu(0.0) == 0.0
    for z in (-20.0, -1.5, 0.3, 4.0, 30.0):
        assert abs(oracle.silu(z) - F.silu(torch.tensor(z, dtype=torch.float64)).item()) < 1e-14
    assert abs(oracle.silu(40.0) - 40.0) < 1e-12 and abs(oracle.silu(-40.0)) < 1e-12


def test_rope_closed_forms(oracle):
    rng = np.random.default_rng(2)
    d, theta = 64, 1e4
    q, k = rng.standard_normal(d), rng.standard_normal(d)
    assert np.array_equal(oracle.rope(q, 0, theta), q)                                  # R_0 = I
    assert abs(np.linalg.norm(oracle.rope(q, 1234, theta)) - np.linalg.norm(q)) < 1e-12   # rotation
    # relative-position property: <R_m q, R_n k> = <R_{m-n} q, k>
    for m, n in ((17, 5), (900, 899), (3, 40)):
        lhs = oracle.rope(q, m, theta) @ oracle.rope(k, n, theta)
        if m >= n:
            rhs = oracle.rope(q, m - n, theta) @ k
        else:
            rhs = q @ oracle.rope(k, n - m, theta)
        assert abs(lhs - rhs) < 1e-9
    # pair (i, i + d/2) is the complex number x_i + j x_{i+d/2} multiplied by exp(j p theta^(-2i/d))
    p = 77
    z = (q[: d // 2] + 1j * q[d // 2:]) * np.exp(1j * p * theta ** (-2.0 * np.arange(d // 2) / d))
    got = oracle.rope(q, p, theta)
    assert np.allclose(got[: d // 2], z.real, atol=1e-12) and np.allclose(got[d // 2:], z.imag, atol=1e-12)
    # first pair turns by exactly p radians, whatever theta is
    e = np.zeros(d); e[0] = 1.0
    r = oracle.rope(e, 1, 1e6)
    assert abs(r[0] - math.cos(1.0)) < 1e-15 and abs(r[d // 2] - math.sin(1.0)) < 1e-15


def test_attention_against_library_and_special_cases(oracle):
    rng = np.random.default_rng(3)
    n, d = 37, 16
    q, k, v = rng.standard_normal(d), rng.standard_normal((n, d)), rng.standard_normal((n, d))
    want = F.scaled_dot_product_attention(torch.from_numpy(q)[None, None, None], torch.from_numpy(k)[None, None],
                                          torch.from_numpy(v)[None, None])[0, 0, 0].numpy()
    assert np.allclose(oracle.attend(q, k, v), want, atol=1e-13)
    # identical keys -> plain average of the values
    same = np.tile(k[:1], (n, 1))
    assert np.allclose(oracle.attend(q, same, v), v.mean(0), atol=1e-13)
    # one overwhelming key -> its value
    big = k.copy(); big[5] = 200.0 * q
    assert np.allclose(oracle.attend(q, big, v), v[5], atol=1e-9)
    # constant values come back unchanged (weights sum to one), even for huge scores
    assert np.allclose(oracle.attend(1e3 * q, k, np.ones((n, d))), 1.0, atol=1e-12)
    # the scale is 1/sqrt(d): two keys, scores s0, s1 -> weight of key 0 is a logistic of (s0-s1)/sqrt(d)
    k2 = rng.standard_normal((2, d)); v2 = np.stack([np.ones(d), np.zeros(d)])
    w0 = 1.0 / (1.0 + math.exp(-(q @ k2[0] - q @ k2[1]) / math.sqrt(d)))
    assert np.allclose(oracle.attend(q, k2, v2), w0, atol=1e-13)


def test_argmax_ties_and_margin(oracle):
    z = np.array([0.5, 2.0, -1.0, 2.0, 1.5])
    assert oracle.argmax(z) == (1, 0.0)                 # lowest id wins a tie
    assert oracle.argmax(z, limit=1) [0] == 0
    z2 = np.array([0.5, 2.0, -1.0, 2.25, 1.5])
    i, m = oracle.argmax(z2)
    assert i == 3 and abs(m - 0.25) < 1e-15
    assert oracle.argmax(z2, limit=3) == (1, 1.5)       # ids >= limit are never chosen
