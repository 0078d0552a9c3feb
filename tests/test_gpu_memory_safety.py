"""Memory safety and resume through the C ABI.

Guard bands: every bound array sits between canary regions in one big allocation; after init, steps (single and
fused, both gradient points, with and without the observer) every canary and every padding column must be
untouched, for each kernel variant at sizes whose tiles are ragged in both directions.

Resume: the state is (x, y, g, step counter); the noise is a pure function of (seed, step, worker, coordinate), so
a run that is stopped, copied out and continued in a fresh state reproduces the uninterrupted run bit for bit.
"""
import numpy as np
import pytest

from oracle import detag_oracle as orc
from paper_2006_08085_b200 import binding as B
from paper_2006_08085_b200 import build, inputs
from paper_2006_08085_b200.session import Session

pytestmark = pytest.mark.gpu
CANARY = 12345.5
GUARD = 1024  # floats on each side of every array


@pytest.fixture(scope="module", autouse=True)
def _built():
    build.build()


def _guarded_state(torch, m, d, ld, K, eta, observe, variant, where):
    n = m.n
    names = ["x", "y", "g", "a", "c"] + (["obs"] if observe else [])
    span = n * ld + 2 * GUARD
    span += (-span) % 4  # keep every array 16-byte aligned
    pool = torch.full((span * len(names),), CANARY, dtype=torch.float32, device="cuda:0")
    views = {}
    for k, name in enumerate(names):
        flat = pool[k * span + GUARD: k * span + GUARD + n * ld]
        views[name] = flat.view(n, ld)
    st = B.detag_create(n, d, m.row_ptr, m.col_idx, m.vals, K, eta, 0.05)
    ws = torch.zeros(B.detag_workspace_bytes(st) + 256, dtype=torch.uint8, device="cuda:0")
    wsp = ws.data_ptr() + (-ws.data_ptr()) % 256
    B.detag_bind(st, ld, views["x"], views["y"], views["g"], views["a"], views["c"], wsp, ws.numel() - 256)
    B.detag_set_noise(st, 0.1, 3, 0)
    B.detag_set_variant(st, variant)
    B.detag_set_gradient_point(st, where)
    if observe:
        B.detag_observe_gossiped_tracker(st, views["obs"])
    return st, pool, views, names, span, ws


@pytest.mark.parametrize("n,d,ld,K,variant", [
    (5, 30, 48, 2, B.DETAG_VARIANT_DENSE), (32, 131, 132, 3, B.DETAG_VARIANT_DENSE), (3, 2, 4, 1, B.DETAG_VARIANT_DENSE),
    (33, 67, 68, 2, B.DETAG_VARIANT_DENSE), (50, 130, 136, 3, B.DETAG_VARIANT_DENSE), (64, 65, 68, 2, B.DETAG_VARIANT_DENSE),
    (64, 67, 72, 4, B.DETAG_VARIANT_RING), (96, 130, 132, 2, B.DETAG_VARIANT_RING),
    (64, 67, 72, 4, B.DETAG_VARIANT_TORUS), (32, 130, 132, 2, B.DETAG_VARIANT_TORUS), (64, 3, 4, 2, B.DETAG_VARIANT_TORUS),
    (72, 67, 68, 2, B.DETAG_VARIANT_DENSE), (100, 130, 132, 3, B.DETAG_VARIANT_DENSE), (128, 31, 32, 2, B.DETAG_VARIANT_DENSE),
    (9, 77, 80, 3, B.DETAG_VARIANT_CSR), (70, 33, 36, 2, B.DETAG_VARIANT_CSR)])
def test_nothing_outside_the_arrays_is_written(n, d, ld, K, variant):
    import torch

    rng = np.random.default_rng(n * 7 + d)
    graph = inputs.torus_graph(n // 8, 8) if variant == B.DETAG_VARIANT_TORUS else inputs.ring_graph(n)
    m = inputs.metropolis_weights(graph)
    eta = orc.spectrum(m.to_dense()).eta
    for where in (B.DETAG_GRADIENT_AT_NEW_MODEL, B.DETAG_GRADIENT_AT_PHASE_START):
        for observe in (False, True):
            st, pool, views, names, span, ws = _guarded_state(torch, m, d, ld, K, eta, observe, variant, where)
            try:
                views["a"][:, :d] = torch.from_numpy(rng.uniform(0.5, 2.0, (n, d)).astype(np.float32))
                views["c"][:, :d] = torch.from_numpy(rng.standard_normal((n, d)).astype(np.float32))
                views["x"][:, :d] = torch.from_numpy(rng.standard_normal((n, d)).astype(np.float32))
                B.detag_init(st)
                B.detag_step(st)
                B.detag_step_many(st, 3)
                B.detag_step(st)
                B.detag_consensus_error(st)
                B.detag_status(st)
                torch.cuda.synchronize()
                for k, name in enumerate(names):
                    lo = pool[k * span: k * span + GUARD]
                    hi = pool[k * span + GUARD + n * ld: (k + 1) * span]
                    assert bool((lo == CANARY).all()) and bool((hi == CANARY).all()), (name, where, observe)
                    assert bool((views[name][:, d:] == CANARY).all()), (name, "padding columns", where, observe)
                for name in ("x", "y", "g"):
                    assert bool(torch.isfinite(views[name][:, :d]).all())
            finally:
                B.detag_destroy(st)


@pytest.mark.parametrize("n,d,K", [(16, 5_003, 4), (64, 700, 3), (128, 130, 2), (90, 203, 3)])
def test_resume_is_bit_exact(n, d, K):
    rng = np.random.default_rng(n + d)
    m = inputs.metropolis_weights(inputs.ring_graph(n) if n != 90 else inputs.path_graph(n))
    eta = orc.spectrum(m.to_dense()).eta
    a = rng.uniform(0.5, 2.0, (n, d)).astype(np.float32)
    c = rng.standard_normal((n, d)).astype(np.float32)
    x0 = rng.standard_normal((n, d)).astype(np.float32)
    with Session(m, d, K, eta, 0.05, a, c, x0, 0.1, 6, coord_offset=77) as s:
        s.init()
        s.step(4)
        saved = {k: s.download(k) for k in ("x", "y", "g")}
        t = B.detag_get_step(s.state)
        s.step(5)
        s.status()
        full = {k: s.download(k) for k in ("x", "y", "g")}
    with Session(m, d, K, eta, 0.05, a, c, saved["x"], 0.1, 6, coord_offset=77) as s:
        s.upload("y", saved["y"])
        s.upload("g", saved["g"])
        B.detag_set_step(s.state, t)
        s.step(5)
        s.status()
        for k in ("x", "y", "g"):
            assert np.array_equal(s.download(k), full[k]), k
