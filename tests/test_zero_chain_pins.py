"""Pins of the zero-chain oracle (proof of Theorem 1) against numerical integration, finite differences, closed
forms and the four properties the paper prints for the function."""
import math

import numpy as np
import pytest
import scipy.integrate

from conftest import read_golden
from oracle import zero_chain as zc


def test_phi_is_the_scaled_normal_integral_and_psi_the_printed_bump():
    for z in (-3.0, -0.4, 0.0, 0.7, 2.5):
        want, _ = scipy.integrate.quad(lambda t: math.exp(-0.5 * t * t), -np.inf, z)
        assert zc.phi(np.array([z]))[0] == pytest.approx(math.sqrt(math.e) * want, rel=1e-10)
    assert zc.psi(np.array([0.5, 0.2, -1.0])).tolist() == [0.0, 0.0, 0.0]
    assert zc.psi(np.array([1.0]))[0] == 1.0  # exp(1 - 1/1)
    assert zc.psi(np.array([0.75]))[0] == pytest.approx(math.exp(1 - 4.0), rel=1e-14)


def test_gradient_matches_finite_differences_of_the_value():
    rng = np.random.default_rng(0)
    x = rng.uniform(-1.5, 1.5, (3, 7))
    g = zc.gradient(x)
    h = 1e-6
    for j in range(7):
        e = np.zeros_like(x)
        e[:, j] = h
        fd = (zc.value(x + e) - zc.value(x - e)) / (2 * h)
        assert np.allclose(g[:, j], fd, rtol=1e-6, atol=1e-7), j


def test_value_and_gradient_at_the_origin_in_closed_form():
    T = 9
    x = np.zeros((1, T))
    assert zc.value(x)[0] == pytest.approx(-math.sqrt(2 * math.pi * math.e) / 2, rel=1e-14)  # -Psi(1) Phi(0)
    g = zc.gradient(x)[0]
    assert g[0] == pytest.approx(-math.sqrt(math.e), rel=1e-14)  # -Psi(1) Phi'(0)
    assert np.all(g[1:] == 0.0)


def test_zero_chain_property_and_the_printed_bounds():
    delta0, l1, g_inf, g_min = (float(v) for v in read_golden("zero_chain_constants.txt")[0])
    rng = np.random.default_rng(1)
    T = 12
    for trial in range(200):
        k = int(rng.integers(0, T))  # progress so far
        x = np.zeros((1, T))
        x[0, :k] = rng.uniform(-2.0, 2.0, k) * rng.choice([1.0, 1.0, 0.2], k)
        if k:
            x[0, k - 1] = x[0, k - 1] or 0.3
        g = zc.gradient(x)
        assert zc.prog(g)[0] <= zc.prog(x)[0] + 1          # one more coordinate per gradient at most
        assert np.abs(g).max() <= g_inf                     # G_inf = 23
        assert np.abs(g).max() >= g_min                     # unfinished chain: a gradient entry of size >= 1
        # the start point is at most Delta_0 T above anything the function reaches (its gap to the infimum)
        assert zc.value(np.zeros((1, T)))[0] - zc.value(x)[0] <= delta0 * T
    # l_1-smoothness on random pairs
    a, b = rng.uniform(-2, 2, (500, T)), rng.uniform(-2, 2, (500, T))
    num = np.linalg.norm(zc.gradient(a) - zc.gradient(b), axis=1)
    assert np.all(num <= l1 * np.linalg.norm(a - b, axis=1))


def test_bernoulli_oracle_is_unbiased_and_touches_only_coordinates_beyond_the_progress():
    rng = np.random.default_rng(2)
    n, T, p, lam, gain = 6, 8, 0.25, 0.5, 3.0
    x = np.zeros((n, T))
    x[:, :3] = rng.uniform(0.3, 1.0, (n, 3))
    exact = gain * zc.gradient(x / lam)
    seen = set()
    acc = np.zeros_like(exact)
    reps = 4000
    for t in range(reps):
        g = zc.stochastic_gradient(x, lam, gain, p, seed=11, t=t)
        assert np.array_equal(g[:, :3], exact[:, :3])  # coordinates already reached: exact
        ratio = g[:, 3] / exact[:, 3]
        seen.update(np.round(ratio, 12).tolist())
        acc += g
    assert seen == {0.0, 1.0 / p}  # z / p with z in {0, 1}
    assert np.allclose(acc[:, 3] / reps, exact[:, 3], rtol=0.1)
    z = np.stack([zc.bernoulli_draws(11, t, n, p) for t in range(reps)])
    assert abs(z.mean() - p) < 0.01 and abs(np.corrcoef(z[:, 0], z[:, 1])[0, 1]) < 0.05
    assert np.array_equal(zc.stochastic_gradient(x, lam, gain, 1.0, 5, 1), exact)  # p = 1: the exact gradient
