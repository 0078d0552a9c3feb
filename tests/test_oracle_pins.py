"""Pins of the float64 oracle against what the paper and the mathematics fix.

None of these re-types an oracle formula: each compares the oracle with a closed form,
a library routine, brute force, an invariant, or a value the paper prints.
"""
import math

import numpy as np
import pytest
import scipy.special
import scipy.stats

from conftest import read_golden
from oracle import detag_oracle as orc
from oracle.philox import philox4x32_10
from paper_2006_08085_b200 import inputs


def _csr(w):
    return w.row_ptr, w.col_idx, w.vals


def _problem(w, K, eta, alpha, a, c, sigma=0.0, seed=0, j0=0):
    return orc.Problem(w.row_ptr, w.col_idx, w.vals, K, eta, alpha, a, c, sigma, seed, j0)


# ----------------------------------------------------------------------------- generator
def test_philox_known_answers():
    for row in read_golden("philox4x32_10_kat.txt"):
        v = [int(t, 16) for t in row]
        got = philox4x32_10([v[0]], [v[1]], [v[2]], [v[3]], v[4], v[5])
        assert [int(g[0]) for g in got] == v[6:10]


def test_noise_is_standard_normal_and_independent():
    xi = orc.standard_normal_noise(seed=7, t=3, n=8, j0=1000, j1=1000 + 125_000)  # 1e6 draws
    flat = xi.ravel()
    assert abs(flat.mean()) < 4e-3 and abs(flat.var() - 1.0) < 6e-3
    assert abs(scipy.stats.skew(flat)) < 1e-2 and abs(scipy.stats.kurtosis(flat)) < 2e-2
    assert scipy.stats.kstest(flat[:200_000], "norm").pvalue > 1e-3
    # every worker row separately (catches a wrong cos/sin or pair assignment)
    for i in range(8):
        assert scipy.stats.kstest(xi[i], "norm").pvalue > 1e-4
    # independence: across workers (incl. the two members of a Box-Muller pair), coordinates, steps
    corr = np.corrcoef(xi)
    assert np.abs(corr - np.eye(8)).max() < 1.5e-2
    assert abs(np.corrcoef(xi[0, :-1], xi[0, 1:])[0, 1]) < 1.5e-2
    xi_next = orc.standard_normal_noise(seed=7, t=4, n=8, j0=1000, j1=1000 + 125_000)
    assert abs(np.corrcoef(xi.ravel(), xi_next.ravel())[0, 1]) < 5e-3
    xi_seed = orc.standard_normal_noise(seed=8, t=3, n=8, j0=1000, j1=1000 + 125_000)
    assert abs(np.corrcoef(xi.ravel(), xi_seed.ravel())[0, 1]) < 5e-3
    # squares uncorrelated inside a pair too (radius shared, angle uniform)
    assert abs(np.corrcoef(xi[0] ** 2, xi[1] ** 2)[0, 1]) < 1.5e-2


def test_box_muller_radius_and_angle_follow_their_uniforms():
    """A pair's radius is the chi-square(2) quantile of u_rad and its angle is 2 pi u_ang (library routines, not the
    oracle's formula): fixes which word feeds which, the 23-bit uniforms and the cos/sin order."""
    seed, t, n, j0, j1 = 21, 5, 8, 4000, 4300
    xi = orc.standard_normal_noise(seed, t, n, j0, j1)
    j = np.arange(j0, j1, dtype=np.uint64)
    for q in range(n // 4):
        r = philox4x32_10(j & np.uint64(0xFFFFFFFF), j >> np.uint64(32), np.uint64(q), np.uint64(t), seed, 0)
        for pair in range(2):
            first, second = xi[4 * q + 2 * pair], xi[4 * q + 2 * pair + 1]
            u_rad = ((r[2 * pair] >> np.uint32(9)).astype(np.float64) + 0.5) / 2.0 ** 23
            u_ang = (r[2 * pair + 1] >> np.uint32(9)).astype(np.float64) / 2.0 ** 23
            assert np.allclose(first ** 2 + second ** 2, scipy.stats.chi2(2).isf(u_rad), rtol=1e-10)
            assert np.allclose(np.mod(np.arctan2(second, first), 2 * math.pi), 2 * math.pi * u_ang, atol=1e-9)


def test_noise_is_a_pure_function_of_its_counter():
    full = orc.standard_normal_noise(5, 2, 6, 0, 300)
    part = orc.standard_normal_noise(5, 2, 6, 100, 260)
    assert np.array_equal(full[:, 100:260], part)
    more_workers = orc.standard_normal_noise(5, 2, 11, 0, 300)
    assert np.array_equal(more_workers[:6], full)


# ----------------------------------------------------------------------------- spectrum, eta
def test_eta_special_values():
    # eta = (1-s)/(1+s), s = sqrt(1-lambda^2): 3-4-5 triangles give rationals
    assert orc.eta_from_lambda(0.0) == 0.0
    assert orc.eta_from_lambda(0.6) == pytest.approx(1.0 / 9.0, rel=1e-14)
    assert orc.eta_from_lambda(0.8) == pytest.approx(0.25, rel=1e-14)
    assert orc.eta_from_lambda(1.0 - 1e-12) == pytest.approx(1.0, abs=1e-5)


def test_spectrum_closed_forms():
    # ring with self weight 1/3: eigenvalues (1 + 2 cos(2 pi m / n)) / 3
    for n in (8, 16, 256):
        sp = orc.spectrum(inputs.metropolis_weights(inputs.ring_graph(n)).to_dense())
        assert sp.lambda2 == pytest.approx((1 + 2 * math.cos(2 * math.pi / n)) / 3, abs=1e-12)
        assert sp.lambda_min == pytest.approx((1 + 2 * math.cos(math.pi)) / 3, abs=1e-12)  # n even: -1/3
        assert sp.lam == pytest.approx(sp.lambda2, abs=1e-12)
    # 8x8 torus, weight 1/5: (1 + 2cos(2 pi p/8) + 2cos(2 pi q/8)) / 5
    sp = orc.spectrum(inputs.metropolis_weights(inputs.torus_graph(8, 8)).to_dense())
    assert sp.lambda2 == pytest.approx((3 + 2 * math.cos(math.pi / 4)) / 5, abs=1e-12)
    assert sp.lambda_min == pytest.approx(-3.0 / 5.0, abs=1e-12)
    # lazy random walk on a path (self loops at the ends): eigenvalues cos(pi m / n)
    n = 12
    p = np.zeros((n, n))
    for i in range(n):
        for j in (i - 1, i + 1):
            p[i, min(max(j, 0), n - 1)] += 0.5
    sp = orc.spectrum(p)
    assert sp.lambda2 == pytest.approx(math.cos(math.pi / n), abs=1e-12)
    # average consensus matrix: lambda = 0, eta = 0
    sp = orc.spectrum(inputs.average_consensus_matrix(7).to_dense())
    assert sp.lam == pytest.approx(0.0, abs=1e-12) and sp.eta == pytest.approx(0.0, abs=1e-12)


def test_spectral_gaps_printed_in_the_paper():
    """16-ring Metropolis + slack matrix: the printed one-digit gaps, and exact linearity in kappa."""
    w0 = inputs.metropolis_weights(inputs.ring_graph(16))
    gap0 = 1.0 - orc.spectrum(w0.to_dense()).lam
    for kappa_s, printed_s in read_golden("fig_spectral_gaps.txt"):
        kappa, printed = float(kappa_s), float(printed_s)
        gap = 1.0 - orc.spectrum(inputs.slack_matrix(w0, kappa).to_dense()).lam
        assert gap == pytest.approx(kappa * gap0, rel=1e-9)  # lambda_i(W_kappa) = kappa*lambda_i(W0) + 1 - kappa
        assert 0.7 * printed <= gap <= 1.4 * printed  # the captions round to one digit


# ----------------------------------------------------------------------------- accelerated gossip
def _poly_coefficients(K, eta):
    """Coefficients (ascending powers) of p_K with p_{-1}=p_0=1, p_{r+1} = (1+eta)*t*p_r - eta*p_{r-1}."""
    P = np.polynomial.polynomial
    prev, cur = np.array([1.0]), np.array([1.0])
    for _ in range(K):
        nxt = P.polysub(P.polymulx(cur) * (1.0 + eta), eta * prev)
        prev, cur = cur, nxt
    return cur


@pytest.mark.parametrize("n,K", [(3, 1), (5, 2), (8, 3), (8, 6), (7, 16)])
def test_ag_equals_polynomial_in_dense_matrix_powers(n, K):
    """K-round AG == sum_k coef_k M^k z, by brute-force dense powers (n <= 8), non-symmetric M."""
    rng = np.random.default_rng(n * 100 + K)
    m = inputs.directed_cycle_blend(n, 0.45, 0.35)  # doubly stochastic, M != M^T
    eta = 0.37
    z = rng.standard_normal((n, 5))
    coef = _poly_coefficients(K, eta)
    dense = m.to_dense()
    expect = sum(ck * np.linalg.matrix_power(dense, k) @ z for k, ck in enumerate(coef))
    got = orc.accelerated_gossip(z, *_csr(m), K, eta)
    assert np.allclose(got, expect, rtol=0, atol=1e-12 * np.abs(expect).max() * max(1, np.abs(coef).sum()))
    # a transposed operand must NOT pass (guards the test itself)
    wrong = sum(ck * np.linalg.matrix_power(dense.T, k) @ z for k, ck in enumerate(coef))
    assert not np.allclose(got, wrong, atol=1e-6)


@pytest.mark.parametrize("K", [1, 2, 5, 16])
def test_ag_chebyshev_closed_form_per_eigenvalue(K):
    """p_K(l) = eta^(K/2) [T_K(x) + (x - sqrt(eta)) U_{K-1}(x)], x = (1+eta) l / (2 sqrt(eta))."""
    w = inputs.metropolis_weights(inputs.torus_graph(3, 4))
    dense = w.to_dense()
    sp = orc.spectrum(dense)
    lam_m, vec = np.linalg.eigh(dense)
    x = (1.0 + sp.eta) * lam_m / (2.0 * math.sqrt(sp.eta))
    assert np.allclose(x, lam_m / sp.lam, atol=1e-12)  # with Algorithm 3's eta the argument is l/lambda
    pk = sp.eta ** (K / 2.0) * (scipy.special.eval_chebyt(K, x)
                                + (x - math.sqrt(sp.eta)) * scipy.special.eval_chebyu(K - 1, x))
    rng = np.random.default_rng(K)
    z = rng.standard_normal((12, 4))
    expect = vec @ (pk[:, None] * (vec.T @ z))
    got = orc.accelerated_gossip(z, *_csr(w), K, sp.eta)
    assert np.allclose(got, expect, atol=1e-12)


def test_ag_first_round_uses_z_minus1_equal_z0():
    """K=1: z_1 = (1+eta) M z_0 - eta z_0 (Algorithm 3 starts with z_{-1} = z_0)."""
    w = inputs.metropolis_weights(inputs.ring_graph(6))
    z = np.arange(12, dtype=np.float64).reshape(6, 2) ** 1.5
    eta = 0.3
    expect = (1 + eta) * w.to_dense() @ z - eta * z
    assert np.allclose(orc.accelerated_gossip(z, *_csr(w), 1, eta), expect, atol=1e-13)


def test_ag_preserves_worker_mean_and_is_linear():
    rng = np.random.default_rng(3)
    w = inputs.metropolis_weights(inputs.random_regular4_graph(10, 5))
    sp = orc.spectrum(w.to_dense())
    z1, z2 = rng.standard_normal((10, 7)), rng.standard_normal((10, 7))
    for K in (1, 4, 9):
        out = orc.accelerated_gossip(z1, *_csr(w), K, sp.eta)
        assert np.allclose(out.sum(axis=0), z1.sum(axis=0), atol=1e-12)
        lin = orc.accelerated_gossip(2.0 * z1 - 3.0 * z2, *_csr(w), K, sp.eta)
        assert np.allclose(lin, 2.0 * out - 3.0 * orc.accelerated_gossip(z2, *_csr(w), K, sp.eta), atol=1e-11)
        # a consensus state is a fixed point
        cons = np.tile(rng.standard_normal((1, 7)), (10, 1))
        assert np.allclose(orc.accelerated_gossip(cons, *_csr(w), K, sp.eta), cons, atol=1e-12)


def test_average_consensus_matrix_averages_in_one_round():
    n = 6
    w = inputs.average_consensus_matrix(n)
    sp = orc.spectrum(w.to_dense())
    z = np.random.default_rng(0).standard_normal((n, 9))
    out = orc.accelerated_gossip(z, *_csr(w), 1, sp.eta)
    assert np.allclose(out, np.tile(z.mean(axis=0), (n, 1)), atol=1e-13)


@pytest.mark.parametrize("n,self_w", [(16, 1.0 / 3.0), (256, 1.0 / 3.0), (9, 0.0), (256, 0.0)])
def test_ring_mode_decay_matches_eigen_analysis(n, self_w):
    """Start in the m=1 Fourier mode of a ring: K rounds scale it by p_K(lambda_1) exactly.

    With zero self weight lambda_1 = cos(2 pi / n); the consensus error then decays by p_K^2.
    """
    m = np.zeros((n, n))
    for i in range(n):
        m[i, i] += self_w
        m[i, (i - 1) % n] += (1 - self_w) / 2
        m[i, (i + 1) % n] += (1 - self_w) / 2
    w = inputs.csr_from_dense(m)
    lam1 = self_w + (1 - self_w) * math.cos(2 * math.pi / n)
    eta = orc.eta_from_lambda(lam1)  # momentum tuned to this mode (lambda_n = -1 for even n, s = 0, is never excited)
    z = np.cos(2 * math.pi * np.arange(n) / n)[:, None] * np.array([[1.0, -2.5]])
    for K in (1, 3, 16):
        x = (1 + eta) * lam1 / (2 * math.sqrt(eta))
        pk = eta ** (K / 2) * (scipy.special.eval_chebyt(K, x) + (x - math.sqrt(eta)) * scipy.special.eval_chebyu(K - 1, x))
        out = orc.accelerated_gossip(z, *_csr(w), K, eta)
        assert np.allclose(out, pk * z, atol=1e-11)
        assert orc.consensus_error(out) == pytest.approx(pk ** 2 * orc.consensus_error(z), rel=1e-9)


# ----------------------------------------------------------------------------- gradient
def test_gradient_is_the_derivative_of_the_objective():
    rng = np.random.default_rng(11)
    a = rng.uniform(0.5, 2.0, (3, 6))
    c = rng.standard_normal((3, 6))
    x = rng.standard_normal((3, 6))

    def f(i, xi):
        return 0.5 * float((a[i] * (xi - c[i]) ** 2).sum())

    g = orc.gradient(x, a, c, 0.0, None)
    h = 1e-6
    for i in range(3):
        for j in range(6):
            e = np.zeros(6)
            e[j] = h
            fd = (f(i, x[i] + e) - f(i, x[i] - e)) / (2 * h)
            assert g[i, j] == pytest.approx(fd, abs=1e-7)


def test_stochastic_gradient_noise_scale_and_unbiasedness():
    n, m = 4, 50_000
    a = np.full((n, m), 1.5)
    c = np.full((n, m), -0.25)
    x = np.full((n, m), 2.0)
    p = orc.Problem(None, None, None, 1, 0.0, 0.0, a, c, 0.1, 9, 0)
    g = orc.stochastic_gradient(p, x, 5)
    resid = g - 1.5 * 2.25
    assert abs(resid.mean()) < 1e-3
    assert resid.std() == pytest.approx(0.1, rel=1e-2)


# ----------------------------------------------------------------------------- the step
def _small_problem(seed, n=8, m=6, K=3, sigma=0.1, graph=None, alpha=0.05):
    rng = np.random.default_rng(seed)
    w = graph if graph is not None else inputs.metropolis_weights(inputs.ring_graph(n))
    n = w.n
    a = rng.uniform(0.5, 2.0, (n, m)).astype(np.float32)
    c = (rng.standard_normal((n, m)) + np.arange(n)[:, None] - n / 2).astype(np.float32)
    eta = orc.spectrum(w.to_dense()).eta
    return _problem(w, K, eta, alpha, a, c, sigma, seed), w


def test_tracker_sum_identities():
    """sum_i y = sum_i (latest folded gradient); mean model follows xbar - alpha*ybar (proof of Theorem 3)."""
    p, _ = _small_problem(1)
    x0 = np.zeros((8, 6))
    s = orc.init_state(p, x0)
    assert np.allclose(s.y.sum(0), s.g_new.sum(0), atol=1e-12)
    for _ in range(6):
        y_fold = orc.folded_tracker(s)
        assert np.allclose(y_fold.sum(0), s.g_new.sum(0), atol=1e-10)
        nxt = orc.step(p, s)
        # after (a),(b): the tracker sums to the gradients folded so far (= g_old after the shift)
        assert np.allclose(nxt.y.sum(0), nxt.g_old.sum(0), atol=1e-10)
        assert np.array_equal(nxt.g_old, s.g_new)
        assert np.allclose(nxt.x.mean(0), s.x.mean(0) - p.alpha * y_fold.mean(0), atol=1e-12)
        s = nxt


def test_dsgt_special_case():
    """K=1, eta=0 reduces to gradient tracking: y' = M(y + dg), x' = M x - alpha y'."""
    p, w = _small_problem(2, K=1)
    p = p._replace(eta=0.0)
    dense = w.to_dense()
    s = orc.init_state(p, np.random.default_rng(0).standard_normal((8, 6)))
    s = orc.step(p, s)
    nxt = orc.step(p, s)
    y_expect = dense @ (s.y + s.g_new - s.g_old)
    x_expect = dense @ s.x - p.alpha * y_expect
    assert np.allclose(nxt.y, y_expect, atol=1e-12) and np.allclose(nxt.x, x_expect, atol=1e-12)


def test_average_consensus_reduces_to_centralized_sgd():
    """W = J/n, noise free: the mean model obeys xbar' = xbar - alpha * mean_i a_i (xbar - c_i) once in consensus."""
    n, m = 5, 4
    w = inputs.average_consensus_matrix(n)
    rng = np.random.default_rng(4)
    a = rng.uniform(0.5, 2.0, (n, m))
    c = rng.standard_normal((n, m))
    p = _problem(w, 1, 0.0, 0.1, a, c, 0.0)
    s = orc.init_state(p, np.zeros((n, m)))
    xbar = np.zeros(m)
    for _ in range(5):
        s = orc.step(p, s)
        xbar = xbar - 0.1 * (a * (xbar[None, :] - c)).mean(0)
        assert np.allclose(s.x, np.tile(xbar, (n, 1)), atol=1e-12)


def test_noise_free_fixed_point():
    """All workers converge to x*_j = sum_i a_ij c_ij / sum_i a_ij and the tracker to zero."""
    p, _ = _small_problem(5, n=8, m=5, K=4, sigma=0.0, alpha=0.1)
    s = orc.run(p, np.zeros((8, 5)), 400)
    a, c = p.a.astype(np.float64), p.c.astype(np.float64)
    xstar = (a * c).sum(0) / a.sum(0)
    assert np.allclose(s.x, np.tile(xstar, (8, 1)), atol=1e-9)
    assert np.abs(orc.folded_tracker(s)).max() < 1e-8


def test_step_is_coordinate_separable():
    """A coordinate sub-range run on its own gives the same numbers (noise counter uses global j)."""
    p, _ = _small_problem(6, m=40)
    x0 = np.random.default_rng(1).standard_normal((8, 40))
    full = orc.run(p, x0, 3)
    sub = orc.run(p._replace(a=p.a[:, 10:25], c=p.c[:, 10:25], j0=10), x0[:, 10:25], 3)
    assert np.array_equal(full.x[:, 10:25], sub.x) and np.array_equal(full.y[:, 10:25], sub.y)


def test_consensus_error_definition():
    x = np.array([[1.0, 2.0], [3.0, 2.0], [5.0, 2.0]])
    assert orc.consensus_error(x) == pytest.approx(8.0)
    assert orc.consensus_error(np.tile(np.arange(4.0), (5, 1))) == 0.0


def test_parity_helper_is_the_same_cycle_cut_elsewhere():
    """The storage convention used on the GPU side (gossip, gradient, then fold) is the oracle's step
    (fold, gossip, gradient) cut at another point: on float32-exact data both give identical numbers."""
    from parity import one_step_from_rounded_state

    rng = np.random.default_rng(0)
    w = inputs.metropolis_weights(inputs.ring_graph(6))
    a = rng.choice([0.5, 1.0, 2.0], (6, 9)).astype(np.float32)
    c = rng.integers(-4, 5, (6, 9)).astype(np.float32)
    x0 = rng.integers(-3, 4, (6, 9)).astype(np.float32)
    p = _problem(w, 3, 0.25, 0.0625, a, c, 0.0)
    (x32, y32, g32), (x1, yg1, g1, yf1) = one_step_from_rounded_state(p, x0)
    s0 = orc.init_state(p, x0)
    assert np.array_equal(x32, s0.x) and np.array_equal(g32, s0.g_new)  # nothing was lost in the rounding
    s1 = orc.step(p, s0)
    assert np.array_equal(s1.x, x1) and np.array_equal(s1.y, yg1) and np.array_equal(s1.g_new, g1)
    assert np.array_equal(orc.folded_tracker(s1), yf1)


# ----------------------------------------------------------------------------- Algorithm 2 with its printed timing
def _dense_polynomial(dense, K, eta):
    """P_K by explicit matrix products (brute force, independent of the oracle's row-wise rounds)."""
    prev = np.eye(dense.shape[0])
    cur = prev.copy()
    for _ in range(K):
        prev, cur = cur, (1.0 + eta) * dense @ cur - eta * prev
    return cur


def test_printed_timing_matches_dense_matrix_recursion():
    """x_{k+1} = P x_k - alpha P y_k, y_{k+1} = P y_k + g(x_k) - g(x_{k-1}) with P from brute-force matrix products."""
    p, w = _small_problem(11, n=8, m=7, K=3, sigma=0.0, alpha=0.03)
    P = _dense_polynomial(w.to_dense(), p.K, p.eta)
    a, c = p.a.astype(np.float64), p.c.astype(np.float64)
    x = np.random.default_rng(2).standard_normal((8, 7))
    g_prev = a * (x - c)
    y = g_prev.copy()
    s = orc.init_phase_state(p, x)
    for _ in range(5):
        g = a * (x - c)  # at the phase-start point
        x, y, g_prev = P @ x - p.alpha * (P @ y), P @ y + g - g_prev, g
        s = orc.phase_as_printed(p, s)
        assert np.allclose(s.x, x, atol=1e-12) and np.allclose(s.y, y, atol=1e-12)
        assert np.allclose(s.g_prev, g_prev, atol=1e-12)


def test_printed_timing_tracker_sum_and_stale_mean_descent():
    """Proof of Theorem 3: mean tracker = mean of the previous phase's gradients; mean model descends along it."""
    p, _ = _small_problem(12, sigma=0.2)
    s = orc.init_phase_state(p, np.random.default_rng(3).standard_normal((8, 6)))
    for _ in range(6):
        assert np.allclose(s.y.sum(0), s.g_prev.sum(0), atol=1e-10)
        nxt = orc.phase_as_printed(p, s)
        assert np.allclose(nxt.x.mean(0), s.x.mean(0) - p.alpha * s.g_prev.mean(0), atol=1e-12)
        # the gradient that entered this phase's fold was taken at the phase-start point, with this phase's noise
        assert np.array_equal(nxt.g_prev, orc.stochastic_gradient(p, s.x, s.t + 1))
        s = nxt


def test_printed_timing_average_consensus_is_delayed_sgd():
    """W = J/n, noise free: xbar_{k+1} = xbar_k - alpha mean_i a_i (x_{k-1,i} - c_i): gradient descent with delay one."""
    n, m, alpha = 5, 4, 0.1
    w = inputs.average_consensus_matrix(n)
    rng = np.random.default_rng(5)
    a = rng.uniform(0.5, 2.0, (n, m))
    c = rng.standard_normal((n, m))
    p = _problem(w, 1, 0.0, alpha, a, c, 0.0)
    s = orc.init_phase_state(p, np.zeros((n, m)))
    x_older = np.zeros(m)  # x_{-1} := x_0 (the initial buffer holds the gradient at x_0)
    x_cur = np.zeros(m)
    for _ in range(6):
        s = orc.phase_as_printed(p, s)
        x_older, x_cur = x_cur, x_cur - alpha * (a * (x_older[None, :] - c)).mean(0)
        assert np.allclose(s.x, np.tile(x_cur, (n, 1)), atol=1e-12)


def test_printed_timing_has_the_same_fixed_point():
    p, _ = _small_problem(13, n=8, m=5, K=4, sigma=0.0, alpha=0.05)
    s = orc.run_as_printed(p, np.zeros((8, 5)), 800)
    a, c = p.a.astype(np.float64), p.c.astype(np.float64)
    xstar = (a * c).sum(0) / a.sum(0)
    assert np.allclose(s.x, np.tile(xstar, (8, 1)), atol=1e-9) and np.abs(s.y).max() < 1e-8


def test_printed_timing_differs_from_the_fresh_gradient_step_only_by_the_gradient_point():
    """Feeding the fresh-gradient step's fold a gradient taken at the old model reproduces the printed phase."""
    p, _ = _small_problem(14, sigma=0.0)
    x0 = np.random.default_rng(6).standard_normal((8, 6))
    s = orc.init_phase_state(p, x0)
    x_new, y_gossip = orc.gossip_and_update(p, s.x, s.y)
    nxt = orc.phase_as_printed(p, s)
    assert np.array_equal(nxt.x, x_new)
    assert np.allclose(nxt.y, orc.fold(y_gossip, orc.gradient(s.x, p.a, p.c, 0.0, None), s.g_prev), atol=1e-13)


# ----------------------------------------------------------------------------- D-PSGD
def test_dpsgd_matches_the_affine_recursion_in_dense_matrix_powers():
    """Noise free, one coordinate at a time the iteration is affine: x' = (P - alpha D_a) x + alpha D_a c with
    P from brute-force matrix products, so x_T = B^T x_0 + (sum_{k<T} B^k) alpha D_a c by explicit powers."""
    p, w = _small_problem(21, n=7, m=5, K=2, sigma=0.0, alpha=0.04)
    P = _dense_polynomial(w.to_dense(), p.K, p.eta)
    x0 = np.random.default_rng(2).standard_normal((7, 5))
    T = 6
    s = orc.run_dpsgd(p, x0, T)
    a, c = p.a.astype(np.float64), p.c.astype(np.float64)
    for j in range(5):
        B = P - p.alpha * np.diag(a[:, j])
        acc = sum(np.linalg.matrix_power(B, k) for k in range(T))
        want = np.linalg.matrix_power(B, T) @ x0[:, j] + acc @ (p.alpha * a[:, j] * c[:, j])
        assert np.allclose(s.x[:, j], want, atol=1e-12)
    assert np.allclose(s.g, a * (s.x - c), atol=1e-12)  # the kept gradient is the one at the current model


def test_dpsgd_plain_form_and_mean_descent():
    """K = 1, eta = 0: x' = M x - alpha g (a non-symmetric M fixes which index of W is summed); the worker
    mean moves by -alpha times the mean gradient because M is doubly stochastic."""
    w = inputs.directed_cycle_blend(6, 0.45, 0.35)
    rng = np.random.default_rng(3)
    a = rng.uniform(0.5, 2.0, (6, 4))
    c = rng.standard_normal((6, 4))
    p = _problem(w, 1, 0.0, 0.07, a, c, 0.2, seed=5)
    s = orc.init_dpsgd_state(p, rng.standard_normal((6, 4)))
    for _ in range(4):
        nxt = orc.dpsgd_step(p, s)
        assert np.allclose(nxt.x, w.to_dense() @ s.x - 0.07 * s.g, atol=1e-13)
        assert np.allclose(nxt.x.mean(0), s.x.mean(0) - 0.07 * s.g.mean(0), atol=1e-13)
        s = nxt


def test_dpsgd_average_consensus_with_equal_curvature_is_centralized_gd_on_the_mean():
    """W = J/n, a_i = a for all workers, noise free: xbar_t = cbar + (1 - alpha a)^t (xbar_0 - cbar), although the
    workers themselves never agree."""
    n, m, alpha = 5, 3, 0.1
    rng = np.random.default_rng(8)
    a = np.tile(rng.uniform(0.5, 2.0, (1, m)), (n, 1))
    c = rng.standard_normal((n, m))
    p = _problem(inputs.average_consensus_matrix(n), 1, 0.0, alpha, a, c, 0.0)
    x0 = rng.standard_normal((n, m))
    s = orc.run_dpsgd(p, x0, 9)
    want = c.mean(0) + (1 - alpha * a[0]) ** 9 * (x0.mean(0) - c.mean(0))
    assert np.allclose(s.x.mean(0), want, atol=1e-13)
    assert orc.consensus_error(s.x) > 1e-4  # non-iid data: D-PSGD's workers stay apart at a constant step size


def test_dpsgd_fixed_point_is_biased_where_detag_is_not():
    """The noise-free D-PSGD limit solves (I - P + alpha D_a) x = alpha D_a c per coordinate (library solve); it is
    not the minimiser of the average objective, which DeTAG reaches on the same problem."""
    p, w = _small_problem(23, n=8, m=4, K=2, sigma=0.0, alpha=0.05)
    P = _dense_polynomial(w.to_dense(), p.K, p.eta)
    a, c = p.a.astype(np.float64), p.c.astype(np.float64)
    s = orc.run_dpsgd(p, np.zeros((8, 4)), 3000)
    for j in range(4):
        want = np.linalg.solve(np.eye(8) - P + p.alpha * np.diag(a[:, j]), p.alpha * a[:, j] * c[:, j])
        assert np.allclose(s.x[:, j], want, atol=1e-9)
    xstar = (a * c).sum(0) / a.sum(0)
    assert np.abs(s.x - xstar[None, :]).max() > 1e-2
    assert np.allclose(orc.run(p, np.zeros((8, 4)), 3000).x, np.tile(xstar, (8, 1)), atol=1e-9)


def test_phase_length_of_theorem_3():
    # sqrt(1 - lambda) = 1/2: R = ln(16) = 2.77 -> 3 rounds; the data-heterogeneity term takes over when it is larger
    assert orc.phase_length(16, 0.75, 0.0, 0.0, 1.0) == 3
    assert orc.phase_length(16, 0.75, 4.0, 1e6, 2.0) == math.ceil(math.log(2e6))  # = ceil(0.5 ln(2e6) / 0.5) = 15
    assert orc.phase_length(2, 0.0, 0.0, 0.0, 1.0) == 1
    # the 256-worker Metropolis ring: lambda = (1 + 2 cos(2 pi/256))/3, R = 0.5 ln 256 / sqrt(1 - lambda) = 195.6
    lam = (1.0 + 2.0 * math.cos(2.0 * math.pi / 256)) / 3.0
    assert orc.phase_length(256, lam, 0.0, 0.0, 1.0) == 196
    # doubling the spectral gap's square root halves the phase
    assert orc.phase_length(1 << 20, 1.0 - 1e-4, 0.0, 0.0, 1.0) == math.ceil(0.5 * math.log(1 << 20) / 1e-2)
