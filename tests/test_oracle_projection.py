"""Pins for oracle/projection.py (Eq. 1 with rotary embedding).  CPU only."""
import numpy as np

from oracle.projection import project_qk, project_v, rope, rope_tables


def test_projection_is_the_matrix_product_of_eq_1():
    rng = np.random.default_rng(0)
    B, n, dm, d, Hq, Hkv = 2, 5, 6, 4, 3, 2
    X = rng.standard_normal((B, n, dm))
    Wq = rng.standard_normal((Hq * d, dm))
    Wk = rng.standard_normal((Hkv * d, dm))
    Q, K = project_qk(X, Wq, Wk, d)
    for b in range(B):
        for t in range(n):
            for h in range(Hq):
                for c in range(d):
                    assert abs(Q[b, h, t, c] - sum(Wq[h * d + c, m] * X[b, t, m] for m in range(dm))) < 1e-12
            for h in range(Hkv):
                for c in range(d):
                    assert abs(K[b, h, t, c] - sum(Wk[h * d + c, m] * X[b, t, m] for m in range(dm))) < 1e-12


def test_value_projection_is_the_matrix_product_of_eq_1():
    rng = np.random.default_rng(5)
    B, n, dm, d, Hkv = 2, 4, 5, 3, 2
    X = rng.standard_normal((B, n, dm))
    Wv = rng.standard_normal((Hkv * d, dm))
    V = project_v(X, Wv, d)
    assert V.shape == (B, Hkv, n, d)
    for b in range(B):
        for t in range(n):
            for h in range(Hkv):
                for c in range(d):
                    assert abs(V[b, h, t, c] - sum(Wv[h * d + c, m] * X[b, t, m] for m in range(dm))) < 1e-12
    # a one-hot X row picks out a column of W_V
    X1 = np.zeros((1, 1, dm)); X1[0, 0, 2] = 1.0
    np.testing.assert_array_equal(project_v(X1, Wv, d)[0, :, 0, :].reshape(-1), Wv[:, 2])


def test_rotation_is_a_complex_multiplication_and_keeps_norms():
    rng = np.random.default_rng(1)
    n, d = 7, 8
    x = rng.standard_normal((2, 3, n, d))
    cos, sin = rope_tables(n, d, theta=100.0)
    y = rope(x, cos.astype(np.float64), sin.astype(np.float64))
    z = (x[..., : d // 2] + 1j * x[..., d // 2:]) * (cos + 1j * sin)
    assert np.allclose(y[..., : d // 2], z.real, atol=1e-12) and np.allclose(y[..., d // 2:], z.imag, atol=1e-12)
    assert np.allclose(np.linalg.norm(y, axis=-1), np.linalg.norm(x, axis=-1), rtol=1e-6)
    assert np.array_equal(rope(x, np.ones((n, d // 2)), np.zeros((n, d // 2))), x)       # angle 0: Eq. 1 as printed
    assert np.array_equal(y[:, :, 0], x[:, :, 0])                                        # token 0 is never turned


def test_tables_follow_the_rotary_schedule():
    cos, sin = rope_tables(16, 8, theta=10000.0)
    assert cos.shape == (16, 4) and cos.dtype == np.float32
    for t in (0, 3, 15):
        for i in range(4):
            ang = t * 10000.0 ** (-2 * i / 8)
            assert abs(cos[t, i] - np.cos(ang)) < 1e-6 and abs(sin[t, i] - np.sin(ang)) < 1e-6
