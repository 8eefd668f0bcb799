"""Pins of the rotary-embedding / cache-append oracle (oracle/rope_oracle.py): properties the
rotation has by construction, an independent complex-number statement, and closed forms."""
import numpy as np

from oracle import rope_oracle as ro


def test_position_zero_is_the_identity_and_rotations_compose():
    rng = np.random.default_rng(0)
    x = rng.standard_normal((5, 64))
    assert np.allclose(ro.rope(x, 0), x, atol=0)
    assert np.allclose(ro.rope(ro.rope(x, 7), 30), ro.rope(x, 37), atol=1e-12)
    assert np.allclose(ro.rope(ro.rope(x, 1234), -1234), x, atol=1e-11)


def test_norms_are_kept_and_scores_depend_on_the_position_difference_only():
    rng = np.random.default_rng(1)
    q, k = rng.standard_normal((2, 128))
    for m, n in ((3, 3), (10, 4), (4096, 4000), (32768, 1)):
        assert np.isclose(np.linalg.norm(ro.rope(q, m)), np.linalg.norm(q), rtol=1e-12)
        for shift in (1, 17, 5000):
            a = ro.rope(q, m) @ ro.rope(k, n)
            b = ro.rope(q, m + shift) @ ro.rope(k, n + shift)
            assert np.isclose(a, b, atol=1e-9)


def test_against_the_complex_number_statement():
    """Pair (x_i, x_{i+D/2}) as the complex number x_i + j x_{i+D/2}, multiplied by exp(j pos theta_i)."""
    rng = np.random.default_rng(2)
    D = 128
    x = rng.standard_normal((3, 7, D))
    pos = rng.integers(0, 40000, (3, 7))
    theta = 10000.0 ** (-np.arange(0, D, 2) / D)
    z = (x[..., :D // 2] + 1j * x[..., D // 2:]) * np.exp(1j * pos[..., None] * theta)
    want = np.concatenate([z.real, z.imag], axis=-1)
    assert np.allclose(ro.rope(x, pos), want, atol=1e-10)


def test_two_features_closed_form_and_a_quarter_turn():
    # D = 2: one pair, theta_0 = 1: a plane rotation by `pos` radians
    x = np.array([1.0, 0.0])
    for pos in (0.0, 1.0, 2.5):
        assert np.allclose(ro.rope(x, pos), [np.cos(pos), np.sin(pos)], atol=1e-15)
    # base = 1: every pair turns by `pos`; pos = pi/2 maps (a, b) to (-b, a)
    y = ro.rope(np.array([1.0, 2.0, 3.0, 4.0]), np.pi / 2, base=1.0)
    assert np.allclose(y, [-3.0, -4.0, 1.0, 2.0], atol=1e-12)


def test_append_places_rows_behind_the_context_and_touches_nothing_else():
    rng = np.random.default_rng(3)
    B, N, Hq, Hkv, D, cap = 3, 5, 4, 2, 8, 20
    q, k, v = rng.standard_normal((B, N, Hq, D)), rng.standard_normal((B, N, Hkv, D)), rng.standard_normal((B, N, Hkv, D))
    kc, vc = rng.standard_normal((B, Hkv, cap, D)), rng.standard_normal((B, Hkv, cap, D))
    pos = rng.integers(0, 100, (B, N))
    kv_len = np.array([0, 15, 16])                     # 16 + 5 > 20: the last sequence does not fit
    q2, k2, v2, st = ro.rope_kv_append(q, k, v, pos, kv_len, kc, vc)
    assert st.tolist() == [0, 0, ro.BAD_LEN]
    assert np.array_equal(k2[2], kc[2]) and np.array_equal(v2[2], vc[2]) and (q2[2] == 0).all()
    for b in (0, 1):
        L = kv_len[b]
        keep = np.ones(cap, bool)
        keep[L:L + N] = False
        assert np.array_equal(k2[b][:, keep], kc[b][:, keep]) and np.array_equal(v2[b][:, keep], vc[b][:, keep])
        for r in range(N):
            assert np.array_equal(v2[b, :, L + r], v[b, r])
            assert np.allclose(k2[b, :, L + r], ro.rope(k[b, r], pos[b, r]), atol=0)
            assert np.allclose(q2[b, r], ro.rope(q[b, r], pos[b, r]), atol=0)
