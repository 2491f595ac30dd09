"""Pins for the oracle's parameter update (Algorithm 1 / 2, line "Update parameters")."""
from fractions import Fraction

import numpy as np

from oracle import uq_oracle as o


def test_printed_update_is_theta_minus_eta_g():
    # dyadic values: every step is exact, so the result is the rational theta - eta * g
    g = np.array([1.5, -2.0, 0.5, -1.0, 1.0, 0.0], dtype=np.float32)     # g_hat of worked example B
    theta = np.array([1.0, 1.0, -3.0, 0.25, 8.0, -0.5], dtype=np.float32)
    new, mom = o.sgd_update(g, theta, None, lr=0.25)
    assert mom is None
    want = [Fraction(float(t)) - Fraction(1, 4) * Fraction(float(x)) for t, x in zip(theta, g)]
    assert [Fraction(float(v)) for v in new] == want
    assert np.array_equal(o.sgd_update(g, theta, None, lr=0.0)[0], theta)


def test_momentum_and_weight_decay_recurrence():
    """Two steps by hand in exact rationals: u = g + wd*theta, buf = mu*buf + u, theta -= lr*buf."""
    lr, mu, wd = Fraction(1, 2), Fraction(1, 4), Fraction(1, 8)
    g1 = np.array([2.0, -4.0, 0.0], dtype=np.float32)
    g2 = np.array([-1.0, 8.0, 0.5], dtype=np.float32)
    theta = np.array([16.0, -8.0, 4.0], dtype=np.float32)
    buf = np.zeros(3, dtype=np.float32)
    th_x = [Fraction(float(t)) for t in theta]
    bf_x = [Fraction(0)] * 3
    for g in (g1, g2):
        theta, buf = o.sgd_update(g, theta, buf, lr=float(lr), mu=float(mu), wd=float(wd))
        for i in range(3):
            u = Fraction(float(g[i])) + wd * th_x[i]
            bf_x[i] = mu * bf_x[i] + u
            th_x[i] = th_x[i] - lr * bf_x[i]
        assert [Fraction(float(v)) for v in theta] == th_x
        assert [Fraction(float(v)) for v in buf] == bf_x


def test_update_matches_float64_within_rounding():
    rng = np.random.default_rng(4)
    g = rng.standard_normal(1000).astype(np.float32) * 1e-2
    theta = rng.standard_normal(1000).astype(np.float32)
    buf = rng.standard_normal(1000).astype(np.float32) * 1e-2
    new, nbuf = o.sgd_update(g, theta, buf, lr=0.1, mu=0.9, wd=5e-4)
    b64 = 0.9 * buf.astype(np.float64) + (g.astype(np.float64) + np.float32(5e-4).astype(np.float64) * theta)
    t64 = theta.astype(np.float64) - np.float64(np.float32(0.1)) * b64
    assert np.allclose(nbuf, b64, rtol=1e-6, atol=1e-9) and np.allclose(new, t64, rtol=1e-6, atol=1e-9)
    # inputs are untouched
    assert np.array_equal(theta, theta.copy())
