"""GPU-vs-oracle parity of Algorithm 2 with the timing it prints (gradient queried at the phase-start point).

Same bars as the default step: one phase from a float32-rounded state, max |err| <= 1e-5 (1 + |ref|) per element
(the stored tracker carries the half-ulp of the stored gradient it telescopes against); trajectories within
1e-4 relative L2 at every phase.
"""
import numpy as np
import pytest

from oracle import detag_oracle as orc
from paper_2006_08085_b200 import binding as B
from paper_2006_08085_b200 import build, inputs
from paper_2006_08085_b200.session import Session
from parity import HALF_ULP32, oracle_problem, rel_l2, worst_ratio

pytestmark = pytest.mark.gpu
AT_START = B.DETAG_GRADIENT_AT_PHASE_START


@pytest.fixture(scope="module", autouse=True)
def _built():
    build.build()


def _check_one_phase(m, K, eta, alpha, a, c, x0, sigma, seed, variants, warm=2, j0=0):
    n, d = a.shape
    p = oracle_problem(m, K, eta, alpha, a, c, sigma, seed, j0)
    s = orc.run_as_printed(p, x0, warm)  # a general state: tracker and gradient buffer differ
    x32, y32, g32 = (v.astype(np.float32) for v in (s.x, s.y, s.g_prev))
    start = orc.PhaseState(x32.astype(np.float64), y32.astype(np.float64), g32.astype(np.float64), s.t)
    ref = orc.phase_as_printed(p, start)
    yg_ref = orc.accelerated_gossip(start.y, m.row_ptr, m.col_idx, m.vals, K, eta)
    for v in variants:
        with Session(m, d, K, eta, alpha, a, c, x32, sigma, seed, coord_offset=j0, observe_gossip=True, variant=v,
                     gradient_point=AT_START) as gpu:
            assert B.detag_get_gradient_point(gpu.state) == AT_START
            gpu.upload("y", y32)
            gpu.upload("g", g32)
            B.detag_set_step(gpu.state, s.t)
            gpu.step()
            gpu.status()
            r = {
                "x": worst_ratio(gpu.download("x"), ref.x),
                "y_gossip": worst_ratio(gpu.download("y_gossip"), yg_ref),
                "g": worst_ratio(gpu.download("g"), ref.g_prev),
                "y": worst_ratio(gpu.download("y"), ref.y, extra=HALF_ULP32 * np.abs(ref.g_prev)),
            }
        assert max(r.values()) <= 1.0, (v, r)


def _check_trajectory(m, K, eta, alpha, a, c, x0, sigma, seed, steps, variants):
    n, d = a.shape
    p = oracle_problem(m, K, eta, alpha, a, c, sigma, seed)
    ref = []
    orc.run_as_printed(p, x0, steps, observe=lambda s: ref.append((s.x.copy(), s.y.copy(), s.g_prev.copy())))
    for v in variants:
        with Session(m, d, K, eta, alpha, a, c, x0, sigma, seed, variant=v, gradient_point=AT_START) as gpu:
            gpu.init()
            for t in range(steps + 1):
                if t > 0:
                    gpu.step()
                errs = {k: rel_l2(gpu.download(k), r) for k, r in zip(("x", "y", "g"), ref[t])}
                if t == 0:
                    errs.pop("x")
                assert max(errs.values()) <= 1e-4, (v, t, errs)
            gpu.status()


def _objective(rng, n, d, scale=1.0):
    a = rng.uniform(0.5, 2.0, (n, d)).astype(np.float32)
    c = (scale * (rng.standard_normal((n, d)) + np.arange(n)[:, None] - n / 2)).astype(np.float32)
    return a, c


@pytest.mark.parametrize("n,d,K", [(5, 37, 2), (8, 301, 3), (12, 1027, 4), (32, 515, 6)])
def test_small_rings_ragged_sizes(n, d, K):
    """n <= 32: the generic rounds kernel and the tensor-core polynomial kernel, several tiles and a ragged tail."""
    rng = np.random.default_rng(n * 100 + d)
    m = inputs.metropolis_weights(inputs.ring_graph(n))
    eta = orc.spectrum(m.to_dense()).eta
    a, c = _objective(rng, n, d)
    x0 = rng.standard_normal((n, d)).astype(np.float32)
    variants = [B.DETAG_VARIANT_CSR, B.DETAG_VARIANT_DENSE]
    _check_one_phase(m, K, eta, 0.05, a, c, x0, 0.1, 13, variants)
    _check_trajectory(m, K, eta, 0.05, a, c, x0, 0.1, 13, 6, variants)


def test_torus_64_dense_polynomial_kernel():
    rng = np.random.default_rng(64)
    m = inputs.gossip_matrix(inputs.CONFIGS["cfg3"])
    eta = orc.spectrum(m.to_dense()).eta
    a, c = _objective(rng, 64, 333, scale=0.2)
    x0 = rng.standard_normal((64, 333)).astype(np.float32)
    _check_one_phase(m, 8, eta, 0.005, a, c, x0, 0.05, 2, [B.DETAG_VARIANT_DENSE, B.DETAG_VARIANT_CSR, B.DETAG_VARIANT_TORUS])
    _check_trajectory(m, 8, eta, 0.005, a, c, x0, 0.05, 2, 5, [B.DETAG_VARIANT_DENSE, B.DETAG_VARIANT_TORUS])


@pytest.mark.parametrize("n,d,K", [(64, 130, 16), (256, 129, 8)])
def test_ring_band_kernel(n, d, K):
    rng = np.random.default_rng(n + d)
    m = inputs.metropolis_weights(inputs.ring_graph(n))
    a, c = _objective(rng, n, d, scale=0.1)
    x0 = rng.standard_normal((n, d)).astype(np.float32)
    _check_one_phase(m, K, 0.3, 0.02, a, c, x0, 0.1, 5, [B.DETAG_VARIANT_RING])
    _check_trajectory(m, K, 0.3, 0.02, a, c, x0, 0.1, 5, 5, [B.DETAG_VARIANT_RING])


@pytest.mark.parametrize("n,d,K", [(100, 131, 4), (72, 64, 3)])
def test_register_resident_dense_kernel(n, d, K):
    rng = np.random.default_rng(n + d)
    m = inputs.metropolis_weights(inputs.random_regular4_graph(n, 3))
    eta = orc.spectrum(m.to_dense()).eta
    a, c = _objective(rng, n, d, scale=0.1)
    x0 = rng.standard_normal((n, d)).astype(np.float32)
    _check_one_phase(m, K, eta, 0.02, a, c, x0, 0.1, 5, [B.DETAG_VARIANT_DENSE, B.DETAG_VARIANT_CSR])
    _check_trajectory(m, K, eta, 0.02, a, c, x0, 0.1, 5, 5, [B.DETAG_VARIANT_DENSE])


def test_first_phase_differs_from_the_default_step_only_in_the_gradient():
    """From the common initial state both gradient points give the same x' (bit for bit); the gradients differ."""
    rng = np.random.default_rng(3)
    m = inputs.metropolis_weights(inputs.ring_graph(8))
    a, c = _objective(rng, 8, 200)
    x0 = rng.standard_normal((8, 200)).astype(np.float32)
    out = {}
    for where in (B.DETAG_GRADIENT_AT_NEW_MODEL, AT_START):
        with Session(m, 200, 3, 0.2, 0.05, a, c, x0, 0.0, 0, gradient_point=where) as gpu:
            gpu.init()
            gpu.step()
            gpu.status()
            out[where] = (gpu.download("x"), gpu.download("g"))
    assert np.array_equal(out[0][0], out[AT_START][0])
    assert np.allclose(out[AT_START][1], a.astype(np.float64) * (x0.astype(np.float64) - c), rtol=1e-6, atol=1e-6)
    assert not np.array_equal(out[0][1], out[AT_START][1])
