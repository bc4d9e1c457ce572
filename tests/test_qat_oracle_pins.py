"""Pins of the QAT-loop oracle (schedule, computed Gaussian table, Adam) against closed forms."""
import numpy as np
from scipy.stats import norm

from oracle import qat_oracle as qo


def test_schedule_end_points_and_constant_ratio():
    T0, Te, N = 1.0, 0.02, 10
    T = [qo.temperature(T0, Te, t, N) for t in range(N + 1)]
    assert T[0] == T0 and abs(T[-1] - Te) < 1e-15
    r = np.array(T[1:]) / np.array(T[:-1])
    np.testing.assert_allclose(r, (Te / T0) ** (1.0 / N), rtol=1e-13)


def test_gaussian_table_inverts_the_normal_cdf_at_cell_centres():
    for Lb in (4, 8, 16):
        S = 1 << Lb
        c = qo.gaussian_codebook(Lb)
        np.testing.assert_allclose(norm.cdf(c), (np.arange(S) + 0.5) / S, rtol=0, atol=1e-13)   # independent routine
        np.testing.assert_allclose(c, -c[::-1], atol=1e-12)                                      # antisymmetric
        assert np.all(np.diff(c) > 0)
    assert abs(qo.gaussian_codebook(16).var() - 1.0) < 1e-3


def test_adam_first_step_and_constant_gradient_closed_forms():
    rng = np.random.default_rng(3)
    p0 = rng.standard_normal(50); g = rng.standard_normal(50) * 10.0 ** rng.integers(-6, 3, 50)
    lr, eps = 1e-3, 1e-8
    p, m, v = qo.adam_update(p0, g, 0.0, 0.0, 1, lr, eps=eps)
    np.testing.assert_allclose(p, p0 - lr * g / (np.abs(g) + eps), rtol=1e-12, atol=0)
    # constant gradient: the bias-corrected moments equal g and g^2 at every step
    m = np.zeros(50); v = np.zeros(50); p = p0.copy()
    for t in range(1, 8):
        p, m, v = qo.adam_update(p, g, m, v, t, lr, eps=eps)
    np.testing.assert_allclose(p, p0 - 7 * lr * g / (np.abs(g) + eps), rtol=1e-10, atol=0)


def test_adam_zero_gradient_and_moment_decay():
    p0 = np.array([1.0, -2.0]); m0 = np.array([0.5, -0.25]); v0 = np.array([4.0, 1.0])
    p, m, v = qo.adam_update(p0, np.zeros(2), m0, v0, 3, 0.1, 0.9, 0.999, 1e-8)
    np.testing.assert_allclose(m, 0.9 * m0); np.testing.assert_allclose(v, 0.999 * v0)
    expect = p0 - 0.1 * (0.9 * m0 / (1 - 0.9 ** 3)) / (np.sqrt(0.999 * v0 / (1 - 0.999 ** 3)) + 1e-8)
    np.testing.assert_allclose(p, expect, rtol=1e-14)
    p, _, _ = qo.adam_update(p0, np.zeros(2), 0.0, 0.0, 1, 0.1)
    np.testing.assert_array_equal(p, p0)


def test_hadamard_matches_scipy_and_is_orthogonal_up_to_its_size():
    from scipy.linalg import hadamard as sp_hadamard
    for n in (1, 2, 8, 64):
        H = qo.hadamard(n)
        np.testing.assert_array_equal(H, sp_hadamard(n))                 # independent construction
        np.testing.assert_array_equal(H @ H, n * np.eye(n))


def test_rotation_is_orthogonal_and_inverts_and_spreads_a_spike():
    rng = np.random.default_rng(8)
    m, n = 16, 32
    W = rng.standard_normal((m, n)); sL = rng.choice([-1.0, 1.0], m); sR = rng.choice([-1.0, 1.0], n)
    Wt = qo.rht_forward(W, sL, sR)
    np.testing.assert_allclose(qo.rht_inverse(Wt, sL, sR), W, atol=1e-13)
    np.testing.assert_allclose(np.linalg.norm(Wt), np.linalg.norm(W), rtol=1e-13)   # Frobenius norm kept
    E = np.zeros((m, n)); E[3, 5] = 1.0                                  # one spike becomes a flat +-1/sqrt(mn) field
    np.testing.assert_allclose(np.abs(qo.rht_forward(E, sL, sR)), 1.0 / np.sqrt(m * n), rtol=1e-13)
    # y = W x  is reproduced from the rotated quantities: (W~ applied to the rotated input)
    x = rng.standard_normal(n)
    xr = qo.hadamard(n) @ (sR * x) / np.sqrt(n)
    back = sL * (qo.hadamard(m) @ (Wt @ xr)) / np.sqrt(m)
    np.testing.assert_allclose(back, W @ x, atol=1e-12)


def test_group_scales_normalise_every_group_of_sixteen():
    rng = np.random.default_rng(9)
    W = rng.standard_normal((4, 64)) * np.array([1.0, 10.0, 0.1, 3.0])[:, None]
    s, Wn = qo.group_scales(W)
    assert s.shape == (4, 4)
    np.testing.assert_allclose((Wn.reshape(4, 4, 16) ** 2).mean(axis=2), 1.0, rtol=1e-13)
    np.testing.assert_allclose(Wn.reshape(4, 4, 16) * s[:, :, None], W.reshape(4, 4, 16), rtol=1e-13)
    np.testing.assert_allclose(qo.group_scales(np.full((1, 16), -2.5))[0], 2.5)
