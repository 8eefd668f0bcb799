"""Pins for the oracle's hidden-transfer projection (Section "Training stage", h~ = W . h)."""
import numpy as np


def test_equals_library_matvec(oracle):
    rng = np.random.default_rng(0)
    B, k, d = 3, 2, 37
    h = rng.standard_normal((B, d)).astype(np.float32)
    W = rng.standard_normal((k, d, d)).astype(np.float32)
    out = oracle.transfer(h, W)
    ref = np.einsum("irc,bc->bir", W.astype(np.float64), h.astype(np.float64))
    assert np.abs(out - ref).max() < 1e-12
    # a transposed operand would give this instead -- it must differ
    wrong = np.einsum("icr,bc->bir", W.astype(np.float64), h.astype(np.float64))
    assert np.abs(out - wrong).max() > 1e-3


def test_identity_and_one_hot(oracle):
    rng = np.random.default_rng(1)
    d = 16
    h = rng.standard_normal((2, d)).astype(np.float32)
    W = np.stack([np.eye(d), np.zeros((d, d))]).astype(np.float32)
    W[1, 3, 11] = 1.0          # output feature 3 of step 2 copies input feature 11
    out = oracle.transfer(h, W)
    assert np.array_equal(out[:, 0], h.astype(np.float64))
    expect = np.zeros((2, d))
    expect[:, 3] = h[:, 11]
    assert np.array_equal(out[:, 1], expect)


def test_linearity_and_step_independence(oracle):
    rng = np.random.default_rng(2)
    d = 24
    h1 = rng.standard_normal((1, d)).astype(np.float32)
    h2 = rng.standard_normal((1, d)).astype(np.float32)
    W = rng.standard_normal((3, d, d)).astype(np.float32)
    a = oracle.transfer(h1, W)
    b = oracle.transfer(h2, W)
    s = oracle.transfer(np.concatenate([h1, h2]), W)
    assert np.array_equal(s[0], a[0]) and np.array_equal(s[1], b[0])
    c = oracle.transfer(2 * h1, W)
    assert np.array_equal(c, 2 * a)
    only2 = oracle.transfer(h1, W[1:2])
    assert np.array_equal(only2[:, 0], a[:, 1])
