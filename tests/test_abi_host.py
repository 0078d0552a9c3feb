"""The C-ABI library: it loads, exports what include/detag.h declares, and its host-only entry points
(spectral routine, argument and CSR validation) behave.  No GPU compute calls here."""
import ctypes
import math
import os
import re

import numpy as np
import pytest

from conftest import ROOT
from paper_2006_08085_b200 import binding as B
from paper_2006_08085_b200 import build, inputs


@pytest.fixture(scope="module", autouse=True)
def _built():
    build.build()


def _declared_symbols():
    text = open(os.path.join(ROOT, "include", "detag.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(detag_[a-z_0-9]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    names = _declared_symbols()
    assert "detag_create" in names and "detag_step" in names and "detag_consensus_error" in names
    assert "detag_destroy" in names and "detag_spectral" in names
    handle = ctypes.CDLL(B.LIB_PATH)
    for name in names:
        assert hasattr(handle, name), name
    assert sorted(B.SIGNATURES) == names  # the binding covers exactly the header


def test_spectral_closed_forms():
    for n in (8, 16, 256):
        w = inputs.metropolis_weights(inputs.ring_graph(n))
        l2, lmin, lam, eta = B.detag_spectral(n, w.row_ptr, w.col_idx, w.vals)
        assert l2 == pytest.approx((1 + 2 * math.cos(2 * math.pi / n)) / 3, abs=1e-12)
        assert lmin == pytest.approx(-1 / 3, abs=1e-12)
        s = math.sqrt(1 - l2 * l2)
        assert lam == pytest.approx(l2, abs=1e-12) and eta == pytest.approx((1 - s) / (1 + s), rel=1e-10)
    w = inputs.metropolis_weights(inputs.torus_graph(8, 8))
    l2, lmin, lam, eta = B.detag_spectral(64, w.row_ptr, w.col_idx, w.vals)
    assert l2 == pytest.approx((3 + math.sqrt(2)) / 5, abs=1e-12) and lmin == pytest.approx(-0.6, abs=1e-12)
    # lambda = 0.6 and 0.8 give eta = 1/9 and 1/4 (3-4-5 triangles): 2x2 blocks [[(1+l)/2,(1-l)/2],...]
    for lam_t, eta_t in ((0.6, 1 / 9), (0.8, 0.25)):
        m = np.array([[(1 + lam_t) / 2, (1 - lam_t) / 2], [(1 - lam_t) / 2, (1 + lam_t) / 2]])
        w = inputs.csr_from_dense(m)
        assert B.detag_spectral(2, w.row_ptr, w.col_idx, w.vals)[3] == pytest.approx(eta_t, rel=1e-12)
    # slack matrix: eigenvalues move linearly in kappa
    w0 = inputs.metropolis_weights(inputs.ring_graph(16))
    g0 = 1 - B.detag_spectral(16, w0.row_ptr, w0.col_idx, w0.vals)[2]
    wk = inputs.slack_matrix(w0, 0.05)
    assert 1 - B.detag_spectral(16, wk.row_ptr, wk.col_idx, wk.vals)[2] == pytest.approx(0.05 * g0, rel=1e-9)
    # average consensus: lambda = 0 -> eta = 0
    w = inputs.average_consensus_matrix(9)
    assert B.detag_spectral(9, w.row_ptr, w.col_idx, w.vals)[2:] == pytest.approx((0.0, 0.0), abs=1e-12)


def test_spectral_errors():
    w = inputs.directed_cycle_blend(5)
    with pytest.raises(B.DetagError) as e:
        B.detag_spectral(5, w.row_ptr, w.col_idx, w.vals)
    assert e.value.code == B.DETAG_ERR_NOT_SYMMETRIC
    # zero-self-weight even ring is bipartite: lambda_n = -1
    m = np.zeros((6, 6))
    for i in range(6):
        m[i, (i - 1) % 6] = m[i, (i + 1) % 6] = 0.5
    w = inputs.csr_from_dense(m)
    with pytest.raises(B.DetagError) as e:
        B.detag_spectral(6, w.row_ptr, w.col_idx, w.vals)
    assert e.value.code == B.DETAG_ERR_SPECTRUM


def _create_code(n, d, rp, ci, va, K=2, eta=0.1, alpha=0.01):
    try:
        st = B.detag_create(n, d, rp, ci, va, K, eta, alpha)
    except B.DetagError as e:
        return e.code
    B.detag_destroy(st)
    return 0


def test_create_validation():
    w = inputs.metropolis_weights(inputs.ring_graph(8))
    assert _create_code(8, 100, w.row_ptr, w.col_idx, w.vals) == 0
    assert _create_code(8, 100, w.row_ptr, w.col_idx, w.vals, eta=float("nan")) == 0
    assert _create_code(8, 0, w.row_ptr, w.col_idx, w.vals) == B.DETAG_ERR_ARG
    assert _create_code(8, 100, w.row_ptr, w.col_idx, w.vals, K=0) == B.DETAG_ERR_ARG
    bad = w.col_idx.copy()
    bad[1] = 99
    assert _create_code(8, 100, w.row_ptr, bad, w.vals) == B.DETAG_ERR_CSR
    bad = w.col_idx.copy()
    bad[0], bad[1] = bad[1], bad[0]
    assert _create_code(8, 100, w.row_ptr, bad, w.vals) == B.DETAG_ERR_CSR
    vals = w.vals.copy()
    vals[0] += 1e-6
    assert _create_code(8, 100, w.row_ptr, w.col_idx, vals) == B.DETAG_ERR_NOT_STOCHASTIC
    # row-stochastic but not column-stochastic
    m = np.array([[0.5, 0.5, 0.0], [0.5, 0.5, 0.0], [0.5, 0.0, 0.5]])
    ws = inputs.csr_from_dense(m)
    assert _create_code(3, 10, ws.row_ptr, ws.col_idx, ws.vals) == B.DETAG_ERR_NOT_STOCHASTIC
    nsym = inputs.directed_cycle_blend(5)
    assert _create_code(5, 10, nsym.row_ptr, nsym.col_idx, nsym.vals, eta=0.2) == 0
    assert _create_code(5, 10, nsym.row_ptr, nsym.col_idx, nsym.vals, eta=float("nan")) == B.DETAG_ERR_NOT_SYMMETRIC


def test_state_accessors_without_device():
    w = inputs.metropolis_weights(inputs.ring_graph(8))
    st = B.detag_create(8, 100, w.row_ptr, w.col_idx, w.vals, 2, float("nan"), 0.05)
    try:
        assert B.detag_workspace_bytes(st) >= 2048 * 8
        assert B.detag_get_step(st) == 0
        B.detag_set_step(st, 7)
        assert B.detag_get_step(st) == 7
        B.detag_set_noise(st, 0.1, 3)
        assert B.detag_get_variant(st) in (B.DETAG_VARIANT_CSR, B.DETAG_VARIANT_DENSE, B.DETAG_VARIANT_RING)
        with pytest.raises(B.DetagError) as e:
            B.detag_step(st)
        assert e.value.code == B.DETAG_ERR_UNBOUND and "bind" in B.detag_last_error(st)
        with pytest.raises(B.DetagError):
            B.detag_set_noise(st, -1.0, 0)
    finally:
        B.detag_destroy(st)


def test_phase_length_matches_theorem_3_and_the_oracle():
    import math

    from oracle import detag_oracle as orc

    lam_ring = (1.0 + 2.0 * math.cos(2.0 * math.pi / 256)) / 3.0
    cases = [(16, 0.75, 0.0, 0.0, 1.0), (16, 0.75, 4.0, 1e6, 2.0), (2, 0.0, 0.0, 0.0, 1.0), (256, lam_ring, 0.0, 0.0, 1.0),
             (64, 0.882843, 9.0, 5e4, 3.0)]
    for case in cases:
        assert B.detag_phase_length(*case) == orc.phase_length(*case), case
    assert B.detag_phase_length(16, 0.75) == 3 and B.detag_phase_length(256, lam_ring) == 196
    for bad in ((0, 0.5), (4, 1.0), (4, -0.1), (4, float("nan"))):
        with pytest.raises(B.DetagError) as e:
            B.detag_phase_length(*bad)
        assert e.value.code == B.DETAG_ERR_ARG


def test_gradient_point_accessors():
    m = inputs.metropolis_weights(inputs.ring_graph(4))
    st = B.detag_create(4, 16, m.row_ptr, m.col_idx, m.vals, 2, 0.1, 0.1)
    try:
        assert B.detag_get_gradient_point(st) == B.DETAG_GRADIENT_AT_NEW_MODEL
        B.detag_set_gradient_point(st, B.DETAG_GRADIENT_AT_PHASE_START)
        assert B.detag_get_gradient_point(st) == B.DETAG_GRADIENT_AT_PHASE_START
        with pytest.raises(B.DetagError) as e:
            B.detag_set_gradient_point(st, 7)
        assert e.value.code == B.DETAG_ERR_ARG
    finally:
        B.detag_destroy(st)
