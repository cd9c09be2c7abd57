"""Pins for the oracle's LAMB direction (Algorithm A2) with the layer-wise update of Eq. upth / Eq. 3."""
import numpy as np
import pytest


def _offs(*sizes):
    return np.concatenate([[0], np.cumsum(sizes)]).astype(np.int64)


def test_first_step_from_zero_moments_is_a_sign_step(oracle):
    """t = 1, m = v = 0, wd = 0, zeta -> 0: m^ = g, v^ = g^2, so u = sign(g) (Adam's first step), ||u_l|| = sqrt(n_l)
    and theta' = theta - lr * tau(||theta_l||) / sqrt(n_l) * sign(g)."""
    offs = _offs(4, 9)
    rng = np.random.RandomState(0)
    theta = rng.randn(13).astype(np.float32)
    g = (rng.randn(13) * 0.3).astype(np.float32)
    z = np.zeros(13, dtype=np.float32)
    th, m, v, norms = oracle.lamb(offs, theta, z, z, g, 1, 0.05, 0.9, 0.999, 1e-30, 0.0)
    assert np.allclose(m, 0.1 * g, rtol=1e-6) and np.allclose(v, 0.001 * g.astype(np.float64) ** 2, rtol=1e-5)
    for l, n in enumerate((4, 9)):
        sl = slice(int(offs[l]), int(offs[l + 1]))
        nt = np.sqrt(np.sum(theta[sl].astype(np.float64) ** 2))
        assert abs(norms[l, 0] - nt) <= 2e-7 * nt and abs(norms[l, 1] - np.sqrt(n)) <= 1e-5
        want = theta[sl] - 0.05 * min(nt, 10.0) / np.sqrt(n) * np.sign(g[sl])
        assert np.allclose(th[sl], want, rtol=2e-5, atol=1e-6)


def test_hand_case(oracle):
    """One layer, theta = (3, 4), m = v = 0, g = (1, -2), beta1 = 0.5, beta2 = 0.75, t = 1, zeta = 1, wd = 0:
    m' = (0.5, -1), v' = (0.25, 1); m^ = (1, -2), v^ = (1, 4); u = (1/2, -2/3); ||u|| = 5/6, ||theta|| = 5;
    theta' = theta - 0.1 * 5 / (5/6) * u = (3 - 0.3, 4 + 0.4) = (2.7, 4.4)."""
    offs = _offs(2)
    theta = np.array([3, 4], dtype=np.float32)
    z = np.zeros(2, dtype=np.float32)
    g = np.array([1, -2], dtype=np.float32)
    th, m, v, norms = oracle.lamb(offs, theta, z, z, g, 1, 0.1, 0.5, 0.75, 1.0, 0.0)
    assert np.array_equal(m, np.array([0.5, -1.0], dtype=np.float32))
    assert np.array_equal(v, np.array([0.25, 1.0], dtype=np.float32))
    assert np.allclose(norms[0], [5.0, 5.0 / 6.0], rtol=1e-6)
    assert np.allclose(th, [2.7, 4.4], rtol=1e-6)


def test_second_step_bias_correction_and_float64_formula(oracle):
    rng = np.random.RandomState(3)
    offs = _offs(300, 5, 1, 77)
    d = int(offs[-1])
    theta = (rng.randn(d) * 0.2).astype(np.float32)
    m0 = (rng.randn(d) * 1e-2).astype(np.float32)
    v0 = (rng.rand(d) * 1e-4).astype(np.float32)
    g = (rng.randn(d) * 1e-2).astype(np.float32)
    b1, b2, zeta, wd, lr, t = 0.9, 0.999, 1e-6, 1e-4, 0.2, 7
    th, m, v, norms = oracle.lamb(offs, theta, m0, v0, g, t, lr, b1, b2, zeta, wd)
    m64 = b1 * m0.astype(np.float64) + (1 - b1) * g
    v64 = b2 * v0.astype(np.float64) + (1 - b2) * g.astype(np.float64) ** 2
    assert np.allclose(m, m64, rtol=1e-6, atol=5e-9) and np.allclose(v, v64, rtol=1e-6, atol=5e-11)
    u = (m64 / (1 - b1 ** t)) / (np.sqrt(v64 / (1 - b2 ** t)) + zeta) + wd * theta
    for l in range(4):
        sl = slice(int(offs[l]), int(offs[l + 1]))
        nt, nu = np.sqrt(np.sum(theta[sl].astype(np.float64) ** 2)), np.sqrt(np.sum(u[sl] ** 2))
        assert np.allclose(norms[l], [nt, nu], rtol=1e-5)
        want = theta[sl] - lr * min(max(nt, 0.0), 10.0) / nu * u[sl]
        assert np.allclose(th[sl], want, rtol=1e-5, atol=1e-7)
        # step length: ||theta' - theta|| = lr * tau(||theta||), whatever the gradient's size
        assert abs(np.sqrt(np.sum((th[sl].astype(np.float64) - theta[sl]) ** 2)) - lr * min(nt, 10.0)) <= 1e-5 * lr * max(nt, 1e-3)


def test_clamp_and_zero_norm_conventions(oracle):
    offs = _offs(2, 3, 2)
    theta = np.array([30, 40, 0, 0, 0, 1, 1], dtype=np.float32)     # ||.|| = 50 -> clipped to c_u; zero tensor -> tau = c_l = 0
    g = np.array([1, 1, 1, 2, 3, 0, 0], dtype=np.float32)           # last layer: zero gradient and zero moments -> u = 0
    z = np.zeros(7, dtype=np.float32)
    th, m, v, norms = oracle.lamb(offs, theta, z, z, g, 1, 0.1, 0.9, 0.999, 1e-6, 0.0, 0.0, 10.0)
    assert abs(np.linalg.norm(th[:2] - theta[:2]) - 0.1 * 10.0) <= 1e-5
    assert np.array_equal(th[2:5], theta[2:5]) and np.all(m[2:5] != 0)          # does not move, moments still update
    assert np.array_equal(th[5:], theta[5:]) and norms[2, 1] == 0.0
    assert np.isfinite(th).all() and np.isfinite(m).all() and np.isfinite(v).all()


def test_inputs_untouched_and_layers_independent(oracle):
    rng = np.random.RandomState(5)
    offs = _offs(10, 20)
    theta, m0, g = [(rng.randn(30) * 0.1).astype(np.float32) for _ in range(3)]
    v0 = (rng.rand(30) * 1e-3).astype(np.float32)
    keep = [a.copy() for a in (theta, m0, v0, g)]
    th, m, v, _ = oracle.lamb(offs, theta, m0, v0, g, 3, 0.1)
    assert all(np.array_equal(a, b) for a, b in zip(keep, (theta, m0, v0, g)))
    th1, m1, v1, _ = oracle.lamb(_offs(10), theta[:10].copy(), m0[:10].copy(), v0[:10].copy(), g[:10].copy(), 3, 0.1)
    assert np.array_equal(th[:10], th1) and np.array_equal(m[:10], m1) and np.array_equal(v[:10], v1)
