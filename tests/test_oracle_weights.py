"""Pins for the oracle's seeded weight generator (CPU only)."""
import os

import numpy as np
import torch

HERE = os.path.dirname(os.path.abspath(__file__))


def _golden_lines(name):
    with open(os.path.join(HERE, "golden", name)) as f:
        return [l.strip() for l in f if l.strip() and not l.startswith("#")]


def test_splitmix64_reference_vector(oracle):
    want = [int(x) for x in _golden_lines("splitmix64_seed1234567.txt")]
    got = [oracle.lib().orc_sm64_nth(1234567, n + 1) for n in range(len(want))]
    assert got == want


def test_bf16_rounding_matches_torch(oracle):
    rng = np.random.default_rng(0)
    x = np.concatenate([
        rng.standard_normal(20000).astype(np.float32) * 0.02,
        # exact ties between two bf16 neighbours, even and odd mantissas
        np.array([1.00390625, 1.01171875, -1.00390625, 3.0517578125e-05 * 1.00390625, 0.0], dtype=np.float32),
    ])
    want = torch.from_numpy(x).to(torch.bfloat16).to(torch.float32).numpy()
    got = np.array([oracle.lib().orc_round_bf16(float(v)) for v in x], dtype=np.float32)
    assert np.array_equal(got.view(np.uint32), want.view(np.uint32))


def test_weight_statistics(oracle):
    w = oracle.fill_tensor(0, 0, 0, 0, 2_000_000).astype(np.float64)
    assert abs(w.mean()) < 5e-5
    assert abs(w.std() / 0.02 - 1.0) < 0.01
    z = w / w.std()
    assert abs((z ** 3).mean()) < 0.01                     # symmetric
    assert abs((z ** 4).mean() - (3.0 - 0.1)) < 0.03       # Irwin-Hall(12): excess kurtosis -6/(5*12)
    assert np.abs(w).max() <= 0.02 * 6.0 + 1e-6            # tails end at six sigma
    # all values are bf16: the low 16 bits of the float are zero
    assert not np.any(oracle.fill_tensor(0, 0, 0, 0, 4096).view(np.uint32) & 0xFFFF)


def test_streams_are_distinct_and_reproducible(oracle):
    a = oracle.fill_tensor(0, 0, 17, 0, 1000)
    assert np.array_equal(a, oracle.fill_tensor(0, 0, 17, 0, 1000))
    assert np.array_equal(a[100:200], oracle.fill_tensor(0, 0, 17, 100, 100))
    for other in (oracle.fill_tensor(1, 0, 17, 0, 1000), oracle.fill_tensor(0, 1, 17, 0, 1000),
                  oracle.fill_tensor(0, 0, 18, 0, 1000)):
        assert abs(np.corrcoef(a, other)[0, 1]) < 0.15
    # neighbouring elements are uncorrelated
    w = oracle.fill_tensor(0, 0, 0, 0, 200_000).astype(np.float64)
    assert abs(np.corrcoef(w[:-1], w[1:])[0, 1]) < 0.01


def test_element_from_published_definition(oracle):
    """One element recomputed with Python integers from the stated construction."""
    M = (1 << 64) - 1
    G = 0x9E3779B97F4A7C15

    def mix(z):
        z = ((z ^ (z >> 30)) * 0xBF58476D1CE4E5B9) & M
        z = ((z ^ (z >> 27)) * 0x94D049BB133111EB) & M
        return z ^ (z >> 31)

    seed, tag, tid, idx = 0, 1, 33, 12345
    key = mix((mix((mix((seed + G) & M) + G + tag) & M) + G + tid) & M)
    assert key == oracle.lib().orc_stream_key(seed, tag, tid)
    S = 0
    for lane in range(3):
        r = mix((key + (3 * idx + lane + 1) * G) & M)
        S += sum((r >> s) & 0xFFFF for s in (0, 16, 32, 48))
    z = np.float32(S - 6 * 65535) / np.float32(65536.0)
    w = torch.tensor(np.float32(0.02) * z).to(torch.bfloat16).to(torch.float32).item()
    assert oracle.fill_tensor(seed, tag, tid, idx, 1)[0] == np.float32(w)
