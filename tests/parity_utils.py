"""Helpers shared by the GPU parity tests."""
import numpy as np

# Tolerances of the parity contract: teacher-forced logits within 0.05 absolute and cosine >= 0.9999;
# greedy tokens must agree wherever the oracle's top-2 margin is at least 0.05.
MAX_ABS = 0.05
MIN_COS = 0.9999
MARGIN = 0.05


def cosine(a, b):
    a = np.asarray(a, dtype=np.float64).ravel()
    b = np.asarray(b, dtype=np.float64).ravel()
    return float(a @ b / (np.linalg.norm(a) * np.linalg.norm(b)))


def assert_logits_close(got, want, what=""):
    got = np.asarray(got, dtype=np.float64)
    want = np.asarray(want, dtype=np.float64)
    assert got.shape == want.shape, (got.shape, want.shape)
    assert np.isfinite(got).all(), f"{what}: non-finite logits"
    err = float(np.abs(got - want).max())
    cos = cosine(got, want)
    assert err <= MAX_ABS and cos >= MIN_COS, f"{what}: max abs err {err:.4g}, cosine {cos:.7f}"
    return err, cos


def shape_dict(shape, **over):
    d = shape.as_dict() if hasattr(shape, "as_dict") else dict(shape)
    d.update(over)
    return d
