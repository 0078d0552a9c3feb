"""GPU-vs-oracle parity through the C ABI (needs a B200).

Bars (floating point): after one step max |err| <= 1e-5 (1 + |ref|) per element; over a trajectory the
relative L2 error of every state array is <= 1e-4 at every step.  The folded tracker the library stores
telescopes against the *stored float32* gradient, so its per-element bound carries that value's
half-ulp, 2^-24 |g'|, on top.
"""
import numpy as np
import pytest

from oracle import detag_oracle as orc
from paper_2006_08085_b200 import binding as B
from paper_2006_08085_b200 import build, inputs
from paper_2006_08085_b200.session import Session
from parity import HALF_ULP32, one_step_from_rounded_state, oracle_problem, rel_l2, worst_ratio

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _built():
    build.build()


def _variants_for(m, K):
    """Every kernel variant that accepts this matrix (CSR always does)."""
    out = [B.DETAG_VARIANT_CSR]
    st = B.detag_create(m.n, 8, m.row_ptr, m.col_idx, m.vals, K, 0.1, 0.1)
    try:
        for v in (B.DETAG_VARIANT_DENSE, B.DETAG_VARIANT_RING, B.DETAG_VARIANT_TORUS):
            try:
                B.detag_set_variant(st, v)
                out.append(v)
            except B.DetagError:
                pass
    finally:
        B.detag_destroy(st)
    return out


def _random_objective(rng, n, d, scale=1.0):
    a = rng.uniform(0.5, 2.0, (n, d)).astype(np.float32)
    c = (scale * (rng.standard_normal((n, d)) + np.arange(n)[:, None] - n / 2)).astype(np.float32)
    return a, c


def _check_one_step(m, K, eta, alpha, a, c, x0, sigma, seed, j0=0, variants=None):
    """One step from the oracle's float32-rounded initial state; every observable per element."""
    n, d = a.shape
    p = oracle_problem(m, K, eta, alpha, a, c, sigma, seed, j0)
    (x32, y32, g32), (x_ref, yg_ref, g_ref, yf_ref) = one_step_from_rounded_state(p, x0)
    worst = {}
    for v in variants or _variants_for(m, K):
        with Session(m, d, K, eta, alpha, a, c, x32, sigma, seed, coord_offset=j0, observe_gossip=True,
                     variant=v) as s:
            s.upload("y", y32)
            s.upload("g", g32)
            B.detag_set_step(s.state, 0)
            s.step()
            s.status()
            r = {
                "x": worst_ratio(s.download("x"), x_ref),
                "y_gossip": worst_ratio(s.download("y_gossip"), yg_ref),
                "g": worst_ratio(s.download("g"), g_ref),
                "y": worst_ratio(s.download("y"), yf_ref, extra=HALF_ULP32 * np.abs(g_ref)),
            }
        assert max(r.values()) <= 1.0, (v, r)
        worst[v] = r
    return worst


def _check_trajectory(m, K, eta, alpha, a, c, x0, sigma, seed, steps, j0=0, variants=None, bound=1e-4):
    """Whole pipeline on the GPU (init + steps) against the pure float64 oracle run, every step."""
    n, d = a.shape
    p = oracle_problem(m, K, eta, alpha, a, c, sigma, seed, j0)
    ref = []
    orc.run(p, x0, steps, observe=lambda s: ref.append((s.x.copy(), orc.folded_tracker(s), s.g_new.copy())))
    for v in variants or _variants_for(m, K):
        with Session(m, d, K, eta, alpha, a, c, x0, sigma, seed, coord_offset=j0, variant=v) as s:
            s.init()
            for t in range(steps + 1):
                if t > 0:
                    s.step()
                errs = {k: rel_l2(s.download(k), r) for k, r in zip(("x", "y", "g"), ref[t])}
                if t == 0:
                    errs.pop("x")  # x0 is an input (and may be all zero)
                assert max(errs.values()) <= bound, (v, t, errs)
            s.status()
            # consensus error = squared norm of the projection of x off the consensus space, so by the
            # triangle inequality its root moves by at most ||x_gpu - x_ref||_F
            ce, ce_ref = s.consensus_error(), orc.consensus_error(ref[-1][0])
            dist = float(np.sqrt(((s.download("x").astype(np.float64) - ref[-1][0]) ** 2).sum()))
            assert abs(np.sqrt(ce) - np.sqrt(ce_ref)) <= dist * (1 + 1e-9) + 1e-12 * np.sqrt(ce_ref)


# ----------------------------------------------------------------------------- small and edge cases
@pytest.mark.parametrize("n,d,K", [(3, 1, 1), (5, 37, 2), (8, 300, 3), (8, 129, 16), (7, 4, 5), (12, 1025, 4),
                                   (33, 130, 2), (40, 257, 3), (50, 64, 4), (63, 67, 5)])
def test_small_rings_ragged_sizes(n, d, K):
    rng = np.random.default_rng(n * 1000 + d)
    m = inputs.metropolis_weights(inputs.ring_graph(n))
    eta = orc.spectrum(m.to_dense()).eta
    a, c = _random_objective(rng, n, d)
    x0 = rng.standard_normal((n, d)).astype(np.float32)
    _check_one_step(m, K, eta, 0.05, a, c, x0, 0.1, 11)
    _check_trajectory(m, K, eta, 0.05, a, c, x0, 0.1, 11, steps=6)


def test_irregular_graph_and_noise_free():
    rng = np.random.default_rng(5)
    m = inputs.metropolis_weights(inputs.path_graph(9))  # degrees 1 and 2
    eta = orc.spectrum(m.to_dense()).eta
    a, c = _random_objective(rng, 9, 77)
    x0 = np.zeros((9, 77), dtype=np.float32)
    _check_one_step(m, 3, eta, 0.05, a, c, x0, 0.0, 0)
    _check_trajectory(m, 3, eta, 0.05, a, c, x0, 0.0, 0, steps=8)


def test_non_symmetric_matrix_is_applied_row_wise():
    rng = np.random.default_rng(6)
    m = inputs.directed_cycle_blend(6, 0.45, 0.35)
    a, c = _random_objective(rng, 6, 50)
    x0 = rng.standard_normal((6, 50)).astype(np.float32)
    _check_one_step(m, 4, 0.3, 0.05, a, c, x0, 0.1, 3)


def test_average_consensus_and_dsgt_special_cases():
    rng = np.random.default_rng(7)
    a, c = _random_objective(rng, 6, 40)
    x0 = rng.standard_normal((6, 40)).astype(np.float32)
    _check_one_step(inputs.average_consensus_matrix(6), 1, 0.0, 0.1, a, c, x0, 0.1, 1)
    _check_one_step(inputs.metropolis_weights(inputs.ring_graph(6)), 1, 0.0, 0.1, a, c, x0, 0.1, 1)  # DSGT


@pytest.mark.parametrize("n,d,K", [(8, 64, 2), (16, 130, 3), (32, 257, 2), (40, 70, 2), (64, 130, 4), (96, 67, 3)])
def test_coordinate_offset_enters_the_noise_counter(n, d, K):
    """Column offsets beyond 2^32 reach the high word of the noise counter in every kernel variant that accepts
    the matrix (each kernel forms coord_offset + j on its own)."""
    rng = np.random.default_rng(8 + n)
    m = inputs.metropolis_weights(inputs.ring_graph(n))
    a, c = _random_objective(rng, n, d, scale=0.2)
    x0 = np.zeros((n, d), dtype=np.float32)
    for j0 in ((1 << 32) + 12345, (5 << 32) - 17):  # the second one crosses a multiple of 2^32 inside the arrays
        _check_one_step(m, K, 0.25, 0.05, a, c, x0, 0.1, 9, j0=j0)


def test_coordinate_offset_in_the_fused_multi_step_call():
    """detag_step_many forms its own noise counters: with an offset beyond 2^32 it must still equal the oracle."""
    rng = np.random.default_rng(21)
    n, d, K, j0 = 16, 1000, 3, (3 << 32) + 999
    m = inputs.metropolis_weights(inputs.ring_graph(n))
    eta = orc.spectrum(m.to_dense()).eta
    a, c = _random_objective(rng, n, d)
    x0 = rng.standard_normal((n, d)).astype(np.float32)
    p = oracle_problem(m, K, eta, 0.05, a, c, 0.1, 4, j0)
    ref = orc.run(p, x0, 6)
    with Session(m, d, K, eta, 0.05, a, c, x0, 0.1, 4, coord_offset=j0) as s:
        assert B.detag_get_variant(s.state) == B.DETAG_VARIANT_DENSE
        s.init()
        s.step_many(6)
        s.status()
        for k, want in (("x", ref.x), ("y", orc.folded_tracker(ref)), ("g", ref.g_new)):
            assert rel_l2(s.download(k), want) <= 1e-4, k
        # noise is what distinguishes offsets: the same run at offset 0 must differ
        got_g = s.download("g")
    with Session(m, d, K, eta, 0.05, a, c, x0, 0.1, 4, coord_offset=j0 - (3 << 32)) as s:
        s.init()
        s.step_many(6)
        assert not np.array_equal(s.download("g"), got_g)


def test_padded_leading_dimension_is_left_untouched():
    rng = np.random.default_rng(9)
    m = inputs.metropolis_weights(inputs.ring_graph(5))
    a, c = _random_objective(rng, 5, 30)
    for v in _variants_for(m, 2):
        with Session(m, 30, 2, 0.2, 0.05, a, c, np.zeros((5, 30), np.float32), 0.1, 1, ld=48, variant=v) as s:
            for t in (s.x, s.y, s.g):
                t[:, 30:] = 777.0
            s.init()
            s.step(3)
            s.status()
            for t in (s.x, s.y, s.g):
                assert bool((t[:, 30:] == 777.0).all())


def test_large_worker_count_n_256_and_n_1000():
    rng = np.random.default_rng(10)
    for n, d, K in ((256, 70, 3), (1000, 9, 2)):
        m = inputs.metropolis_weights(inputs.ring_graph(n))
        a, c = _random_objective(rng, n, d, scale=0.05)
        x0 = np.zeros((n, d), dtype=np.float32)
        _check_one_step(m, K, 0.4, 0.01, a, c, x0, 0.1, 2)


def test_noise_matches_the_counter_based_definition():
    """a = 0 makes the gradient pure noise: g = sigma * xi.  Float32 elementary functions on the device
    against the float64 transform: absolute error of a standard normal below 6e-6 everywhere, 1e-6 rms."""
    n, d = 12, 50_000
    m = inputs.metropolis_weights(inputs.ring_graph(n))
    zeros = np.zeros((n, d), dtype=np.float32)
    for v in _variants_for(m, 1):
        with Session(m, d, 1, 0.0, 0.0, zeros, zeros, zeros, 1.0, 77, coord_offset=999, variant=v) as s:
            s.init()
            for t in range(2):
                if t:
                    s.step()
                ref = orc.standard_normal_noise(77, t, n, 999, 999 + d)
                err = s.download("g").astype(np.float64) - ref
                assert np.abs(err).max() < 6e-6 and np.sqrt((err ** 2).mean()) < 1e-6, (v, t, np.abs(err).max())


@pytest.mark.parametrize("n,d,K,kind", [(64, 130, 16, "ring"), (96, 67, 5, "ring"), (64, 200, 4, "directed"),
                                         (128, 64, 8, "two_hop"), (256, 129, 16, "slack"), (512, 70, 8, "ring"),
                                         (1024, 33, 4, "ring")])
def test_circulant_band_variant(n, d, K, kind):
    """Circulant matrices take the banded-polynomial kernel: symmetric ring, a NON-symmetric circulant (fixes the
    sign of the band offset), a two-hop circulant (bandwidth 2), and a slack ring."""
    rng = np.random.default_rng(n + d)
    if kind == "ring":
        m = inputs.metropolis_weights(inputs.ring_graph(n))
    elif kind == "slack":
        m = inputs.slack_matrix(inputs.metropolis_weights(inputs.ring_graph(n)), 0.1)
    elif kind == "directed":
        m = inputs.directed_cycle_blend(n, 0.45, 0.35)
    else:
        dense = np.zeros((n, n))
        for i in range(n):
            for off, w in ((0, 0.4), (1, 0.2), (-1, 0.2), (2, 0.1), (-2, 0.1)):
                dense[i, (i + off) % n] += w
        m = inputs.csr_from_dense(dense)
    assert B.DETAG_VARIANT_RING in _variants_for(m, K)
    a, c = _random_objective(rng, n, d, scale=0.1)
    x0 = rng.standard_normal((n, d)).astype(np.float32)
    _check_one_step(m, K, 0.3, 0.02, a, c, x0, 0.1, 5, variants=[B.DETAG_VARIANT_RING])
    _check_trajectory(m, K, 0.3, 0.02, a, c, x0, 0.1, 5, steps=5, variants=[B.DETAG_VARIANT_RING])


def _block_circulant(kind, R):
    """n = 8 R workers in R blocks of 8, block (r, r') a function of |r - r'| on the block cycle only."""
    if kind == "torus":
        return inputs.metropolis_weights(inputs.torus_graph(R, 8))
    n = 8 * R
    dense = np.zeros((n, n))
    shift = np.roll(np.eye(R), 1, axis=1)
    if kind == "anisotropic":  # different weights along the two axes of the torus
        ring8 = np.roll(np.eye(8), 1, axis=1)
        dense = 0.3 * np.eye(n) + 0.25 * np.kron(shift + shift.T, np.eye(8)) + 0.1 * np.kron(np.eye(R), ring8 + ring8.T)
    else:  # "path_blocks": the blocks are NOT circulant (a path inside each block), only the block cycle is
        inner = inputs.metropolis_weights(inputs.path_graph(8)).to_dense()
        dense = 0.6 * np.kron(np.eye(R), inner) + 0.2 * np.kron(shift + shift.T, np.eye(8))
    return inputs.csr_from_dense(dense)


@pytest.mark.parametrize("R,d,K,kind", [(8, 130, 8, "torus"), (4, 67, 3, "torus"), (8, 1, 2, "torus"), (8, 1025, 4, "anisotropic"),
                                         (4, 300, 5, "anisotropic"), (8, 259, 3, "path_blocks"), (4, 64, 6, "path_blocks")])
def test_block_circulant_transform_variant(R, d, K, kind):
    """Tori (uniform and anisotropic weights) and a block-circulant matrix whose blocks are not circulant: the
    transform kernel must give the oracle's rounds, per element and over a trajectory, at ragged sizes."""
    rng = np.random.default_rng(R * 100 + d)
    m = _block_circulant(kind, R)
    n = 8 * R
    assert B.DETAG_VARIANT_TORUS in _variants_for(m, K)
    eta = orc.spectrum(m.to_dense()).eta
    a, c = _random_objective(rng, n, d, scale=0.2)
    x0 = rng.standard_normal((n, d)).astype(np.float32)
    _check_one_step(m, K, eta, 0.02, a, c, x0, 0.1, 5, j0=(1 << 32) + 7, variants=[B.DETAG_VARIANT_TORUS])
    _check_trajectory(m, K, eta, 0.02, a, c, x0, 0.1, 5, steps=6, variants=[B.DETAG_VARIANT_TORUS])


def test_transform_variant_is_refused_without_the_structure():
    for m in (inputs.metropolis_weights(inputs.ring_graph(64)),              # circulant, but blocks at +1 and -1 differ
              inputs.metropolis_weights(inputs.random_regular4_graph(32, 1)),
              inputs.metropolis_weights(inputs.torus_graph(8, 4)),            # blocks of 8 straddle two rows of 4
              inputs.metropolis_weights(inputs.torus_graph(3, 8))):           # n = 24
        assert B.DETAG_VARIANT_TORUS not in _variants_for(m, 3)
    cfg3 = inputs.gossip_matrix(inputs.CONFIGS["cfg3"])
    st = B.detag_create(64, 128, cfg3.row_ptr, cfg3.col_idx, cfg3.vals, 8, 0.3, 0.01)
    try:
        assert B.detag_get_variant(st) == B.DETAG_VARIANT_TORUS  # what AUTO picks for the 8 x 8 torus
    finally:
        B.detag_destroy(st)


@pytest.mark.parametrize("n,d,K,kind", [(128, 130, 20, "ring"), (256, 67, 40, "ring"), (96, 200, 30, "directed"),
                                         (64, 131, 3, "dense_row"), (256, 64, 196, "ring")])
def test_circulant_kernel_with_a_dense_polynomial(n, d, K, kind):
    """Phase lengths beyond K * bandwidth = 16 (Theorem 3's regime: K = 196 on the 256-ring) make P_K(M) a dense
    circulant; the circulant kernel then contracts the whole ring per output block.  Also a circulant M that is
    dense itself.  Ragged d: the last d % 64 columns run through the generic kernel in the same call."""
    rng = np.random.default_rng(n + d + K)
    if kind == "ring":
        m = inputs.metropolis_weights(inputs.ring_graph(n))
    elif kind == "directed":
        m = inputs.directed_cycle_blend(n, 0.45, 0.35)
    else:
        row = rng.uniform(0.0, 1.0, n)
        row /= row.sum()
        m = inputs.csr_from_dense(np.stack([np.roll(row, i) for i in range(n)]))  # a full circulant, not symmetric
    assert B.DETAG_VARIANT_RING in _variants_for(m, K)
    eta = 0.3 if kind != "ring" else orc.spectrum(m.to_dense()).eta
    a, c = _random_objective(rng, n, d, scale=0.1)
    x0 = rng.standard_normal((n, d)).astype(np.float32)
    _check_one_step(m, K, eta, 0.02, a, c, x0, 0.1, 5, j0=(1 << 32) + 3, variants=[B.DETAG_VARIANT_RING])
    _check_trajectory(m, K, eta, 0.02, a, c, x0, 0.1, 5, steps=4, variants=[B.DETAG_VARIANT_RING])


@pytest.mark.parametrize("n,d,K,kind", [(100, 130, 6, "regular4"), (65, 67, 3, "ring"), (72, 1, 2, "regular4"),
                                        (88, 31, 4, "regular4"), (96, 1057, 5, "directed"), (104, 64, 8, "regular4"),
                                        (127, 97, 3, "path"), (128, 160, 12, "regular4")])
def test_dense_polynomial_held_in_registers(n, d, K, kind):
    """64 < n <= 128, any matrix: the polynomial as register-resident warp strips.  Unstructured, non-symmetric and
    irregular matrices, worker counts on and off the 8-row blocks, d below, on and off the 32-column halves the
    kernel takes (the remainder runs on the generic kernel in the same call)."""
    rng = np.random.default_rng(n * 31 + d)
    if kind == "regular4":
        m = inputs.metropolis_weights(inputs.random_regular4_graph(n, n + K))
    elif kind == "ring":
        m = inputs.metropolis_weights(inputs.ring_graph(n))
    elif kind == "path":
        m = inputs.metropolis_weights(inputs.path_graph(n))
    else:
        m = inputs.directed_cycle_blend(n, 0.4, 0.35)
    eta = orc.spectrum(m.to_dense()).eta if kind != "directed" else 0.3
    st = B.detag_create(n, d, m.row_ptr, m.col_idx, m.vals, K, eta, 0.05)
    try:
        picked = B.detag_get_variant(st)
    finally:
        B.detag_destroy(st)
    if kind == "regular4":
        assert picked == B.DETAG_VARIANT_DENSE  # no structure, several rounds: the dense polynomial
    if kind == "path":
        assert picked == B.DETAG_VARIANT_CSR    # three rounds over two neighbours: the sparse rounds are cheaper
    a, c = _random_objective(rng, n, d, scale=0.1)
    x0 = rng.standard_normal((n, d)).astype(np.float32)
    variants = [B.DETAG_VARIANT_DENSE]
    _check_one_step(m, K, eta, 0.02, a, c, x0, 0.1, 23, variants=variants)
    _check_one_step(m, K, eta, 0.02, a, c, x0, 0.1, 23, j0=(3 << 32) - 40, variants=variants)
    _check_trajectory(m, K, eta, 0.02, a, c, x0, 0.1, 23, steps=5, variants=variants)


def test_misuse_is_reported_not_faulted():
    import torch

    m = inputs.metropolis_weights(inputs.ring_graph(4))
    st = B.detag_create(4, 16, m.row_ptr, m.col_idx, m.vals, 2, 0.1, 0.1)
    try:
        buf = torch.zeros(4 * 16 + 64, dtype=torch.float32, device="cuda:0")
        ws = torch.zeros(B.detag_workspace_bytes(st) + 256, dtype=torch.uint8, device="cuda:0")
        wsp = ws.data_ptr() + (-ws.data_ptr()) % 256
        good = buf.data_ptr()
        for args in ((15, good, good, good, good, good, wsp, ws.numel() - 256),  # ld < d
                     (18, good, good, good, good, good, wsp, ws.numel() - 256),  # ld not a multiple of 4
                     (16, good + 4, good, good, good, good, wsp, ws.numel() - 256),  # misaligned
                     (16, good, good, good, good, good, wsp + 8, ws.numel() - 256),  # workspace misaligned
                     (16, good, good, good, good, good, wsp, 64)):  # workspace too small
            with pytest.raises(B.DetagError) as e:
                B.detag_bind(st, *args)
            assert e.value.code == B.DETAG_ERR_ARG
        with pytest.raises(B.DetagError) as e:
            B.detag_consensus_error(st)
        assert e.value.code == B.DETAG_ERR_UNBOUND
    finally:
        B.detag_destroy(st)


def test_paper_experiment_settings():
    """The (eta, R) pairs and ring/slack matrices of the paper's own runs, on the synthetic objective: every
    variant that accepts them, one step per element and a short trajectory.  eta is the paper's tuned value, not
    the one Algorithm 3 derives from lambda."""
    from conftest import read_golden

    for row in read_golden("table_detag_hyperparameters.txt"):
        n, kappa, eta, R = int(row[0]), float(row[1]), float(row[2]), int(row[3])
        m = inputs.slack_matrix(inputs.metropolis_weights(inputs.ring_graph(n)), kappa)
        rng = np.random.default_rng(int(1000 * kappa) + n)
        a, c = _random_objective(rng, n, 1500)
        x0 = (0.01 * rng.standard_normal((1, 1500))).repeat(n, 0).astype(np.float32)
        _check_one_step(m, R, eta, 0.05, a, c, x0, 0.1, 17)
        _check_trajectory(m, R, eta, 0.05, a, c, x0, 0.1, 17, steps=8)


# ----------------------------------------------------------------------------- the five configurations
def _config_case(name, d):
    cfg = inputs.CONFIGS[name]
    cfg = cfg.with_d(min(d, cfg.d))
    m = inputs.gossip_matrix(cfg)
    eta = orc.spectrum(m.to_dense()).eta
    a, c, x0 = inputs.objective_data(cfg)
    return cfg, m, eta, a, c, x0


@pytest.mark.parametrize("name,d", [("cfg1", 4096), ("cfg2", 270_000), ("cfg3", 20_003), ("cfg4", 5_001),
                                    ("cfg5", 40_001)])
def test_config_one_step_per_element(name, d):
    cfg, m, eta, a, c, x0 = _config_case(name, d)
    _check_one_step(m, cfg.K, eta, cfg.alpha, a, c, x0, cfg.sigma, cfg.seed)


@pytest.mark.parametrize("name,d,steps", [("cfg1", 4096, 100), ("cfg2", 30_001, 100), ("cfg3", 3_001, 100),
                                          ("cfg4", 601, 50), ("cfg5", 6_001, 100)])
def test_config_trajectory(name, d, steps):
    cfg, m, eta, a, c, x0 = _config_case(name, d)
    _check_trajectory(m, cfg.K, eta, cfg.alpha, a, c, x0, cfg.sigma, cfg.seed, steps=steps)


def test_consensus_error_matches_definition():
    rng = np.random.default_rng(12)
    m = inputs.metropolis_weights(inputs.ring_graph(16))
    x = (rng.standard_normal((16, 100_003)) * 3 + 50).astype(np.float32)
    a = np.ones_like(x)
    with Session(m, x.shape[1], 2, 0.1, 0.1, a, a, x) as s:
        assert s.consensus_error() == pytest.approx(orc.consensus_error(x), rel=1e-12)
        assert s.consensus_error() == s.consensus_error()  # fixed summation order
    cons = np.tile(rng.standard_normal((1, 1000)).astype(np.float32), (16, 1))
    with Session(m, 1000, 2, 0.1, 0.1, a[:, :1000], a[:, :1000], cons) as s:
        assert s.consensus_error() == 0.0


# ----------------------------------------------------------------------------- full size, bench launch configuration
def _full_size_sampled(name, blocks, steps):
    """The config at its full size and in the launch configuration bench.py times (default variant, no observer).

    The oracle cannot run 8e8 elements, but the step never mixes coordinates: sampled coordinate blocks are
    recomputed by the oracle on their own (global column offset in the noise counter) and compared element by
    element after one step and in relative L2 over the config's trajectory.
    """
    import os

    cfg = inputs.CONFIGS[name]
    m = inputs.gossip_matrix(cfg)
    eta = orc.spectrum(m.to_dense()).eta
    with Session(m, cfg.d, cfg.K, eta, cfg.alpha, None, None, None, cfg.sigma, cfg.seed) as s:
        chunk = 1 << 21
        for j0 in range(0, cfg.d, chunk):  # objective data, chunk by chunk (bounded host memory)
            j1 = min(cfg.d, j0 + chunk)
            a, c, x0 = inputs.objective_data(cfg, j0, j1, threads=min(16, os.cpu_count() or 1))
            for nm, host in (("a", a), ("c", c), ("x", x0)):
                getattr(s, nm)[:, j0:j1].copy_(s.torch.from_numpy(host))
        s.init()
        refs = []
        for (j0, w) in blocks:
            a, c, x0 = inputs.objective_data(cfg, j0, j0 + w)
            p = oracle_problem(m, cfg.K, eta, cfg.alpha, a, c, cfg.sigma, cfg.seed, j0)
            (x32, y32, g32), one = one_step_from_rounded_state(p, x0)
            # the initial state the GPU computed itself, against the oracle's (relative L2: it is rounded storage)
            assert rel_l2(s.g[:, j0:j0 + w].cpu().numpy(), g32.astype(np.float64)) < 1e-6
            for nm, host in (("x", x32), ("y", y32), ("g", g32)):  # same float32 start on both sides
                getattr(s, nm)[:, j0:j0 + w].copy_(s.torch.from_numpy(host))
            traj = []
            orc.run(p, x0, steps, observe=lambda st: traj.append((st.x.copy(), orc.folded_tracker(st), st.g_new.copy())))
            refs.append((j0, w, one, traj))
        for t in range(1, steps + 1):
            s.step()
            for (j0, w, one, traj) in refs:
                got = {k: getattr(s, k)[:, j0:j0 + w].cpu().numpy() for k in ("x", "y", "g")}
                if t == 1:
                    x_ref, _, g_ref, yf_ref = one
                    r = {"x": worst_ratio(got["x"], x_ref), "g": worst_ratio(got["g"], g_ref),
                         "y": worst_ratio(got["y"], yf_ref, extra=HALF_ULP32 * np.abs(g_ref))}
                    assert max(r.values()) <= 1.0, (name, j0, r)
                errs = {k: rel_l2(got[k], ref) for k, ref in zip(("x", "y", "g"), traj[t])}
                assert max(errs.values()) <= 1e-4, (name, j0, t, errs)
        s.status()


def test_cfg5_full_size_sampled_blocks():
    d = inputs.CONFIGS["cfg5"].d
    _full_size_sampled("cfg5", [(0, 512), (64 * 12345 + 8, 300), (d // 2 - 100, 333), (d - 640, 640)], steps=20)


def test_cfg4_full_size_sampled_blocks():
    d = inputs.CONFIGS["cfg4"].d
    _full_size_sampled("cfg4", [(0, 64), (500_001, 50), (d - 40, 40)], steps=50)


def test_cfg3_full_size_sampled_blocks():
    d = inputs.CONFIGS["cfg3"].d
    _full_size_sampled("cfg3", [(0, 128), (7_000_003, 96), (d - 128, 128)], steps=10)


# ----------------------------------------------------------------------------- host-resident stepping
@pytest.mark.parametrize("n,d,K,graph", [(16, 100_003, 4, "ring"), (64, 20_000, 3, "ring"), (9, 5_001, 2, "path"),
                                         (100, 17_003, 2, "path")])
def test_step_host_matches_device_resident_stepping(n, d, K, graph):
    """detag_step_host (state in page-locked host memory, chunked through a device staging area) performs the
    same arithmetic per coordinate as detag_step: bit-identical results, several chunks and a ragged last one."""
    import torch

    rng = np.random.default_rng(n + d)
    adj = inputs.ring_graph(n) if graph == "ring" else inputs.path_graph(n)
    m = inputs.metropolis_weights(adj)
    eta = orc.spectrum(m.to_dense()).eta
    a, c = _random_objective(rng, n, d)
    x0 = rng.standard_normal((n, d)).astype(np.float32)
    with Session(m, d, K, eta, 0.05, a, c, x0, 0.1, 21) as s:
        s.init()
        ld = s.ld
        host = {k: torch.empty((n, ld), dtype=torch.float32).pin_memory() for k in ("x", "y", "g", "a", "c")}
        for k in host:
            host[k].copy_(getattr(s, k))
        torch.cuda.synchronize()
        chunk = 128 * 64  # 8192 coordinates per chunk: d spans many chunks
        nbytes = B.detag_host_staging_bytes(s.state, chunk)
        staging = torch.empty(nbytes + 256, dtype=torch.uint8, device="cuda:0")
        sptr = staging.data_ptr() + (-staging.data_ptr()) % 256
        for step in range(3):
            B.detag_set_step(s.state, step)
            B.detag_step_host(s.state, ld, host["x"], host["y"], host["g"], host["a"], host["c"], sptr, nbytes,
                              s.stream())
            B.detag_set_step(s.state, step)
            s.step()
            torch.cuda.synchronize()
            for k in ("x", "y", "g"):
                assert torch.equal(host[k][:, :d], getattr(s, k)[:, :d].cpu()), (k, step)
