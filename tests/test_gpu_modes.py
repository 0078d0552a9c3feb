"""GPU-vs-oracle parity of the two other step modes through the C ABI (needs a B200).

Caller-written gradients: the oracle's step with its gradient evaluation replaced by arrays drawn here and fed
to both sides (Algorithm 2 without the oracle query).  D-PSGD: the oracle's `dpsgd_step`.  Bars as for the
default step: per element max |err| <= 1e-5 (1 + |ref|) after one step from the same float32 state, relative
L2 <= 1e-4 at every step of a trajectory.
"""
import numpy as np
import pytest

from oracle import detag_oracle as orc
from paper_2006_08085_b200 import binding as B
from paper_2006_08085_b200 import build, inputs
from paper_2006_08085_b200.session import Session
from parity import oracle_problem, rel_l2, worst_ratio

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _built():
    build.build()


def _graph(kind, n):
    if kind == "ring":
        return inputs.metropolis_weights(inputs.ring_graph(n))
    if kind == "path":
        return inputs.metropolis_weights(inputs.path_graph(n))
    if kind == "regular4":
        return inputs.metropolis_weights(inputs.random_regular4_graph(n, 4))
    if kind == "directed":
        return inputs.directed_cycle_blend(n, 0.45, 0.35)
    raise ValueError(kind)


def _variants(n, dpsgd_ring=False):
    out = [B.DETAG_VARIANT_CSR] + ([B.DETAG_VARIANT_DENSE] if n <= 32 else [])
    if dpsgd_ring and n >= 64 and n % 32 == 0:
        out.append(B.DETAG_VARIANT_RING)  # the circulant kernel also runs D-PSGD
    return out


# ----------------------------------------------------------------------------- caller-written gradients
@pytest.mark.parametrize("n,d,K,kind", [(8, 300, 3, "ring"), (32, 1027, 6, "regular4"), (5, 37, 2, "path"),
                                         (6, 50, 4, "directed"), (3, 1, 1, "ring"), (40, 130, 2, "ring"),
                                         (64, 67, 3, "ring")])
def test_external_gradients_ten_steps(n, d, K, kind):
    """Both sides get the same externally drawn gradients (large next to the model, so the tracker update
    cancels digits); every step is compared per element from the oracle's float32-rounded previous state, and
    the GPU's own trajectory in relative L2."""
    rng = np.random.default_rng(n * 131 + d)
    m = _graph(kind, n)
    eta = 0.3 if kind == "directed" else orc.spectrum(m.to_dense()).eta
    alpha = 0.02
    x0 = rng.standard_normal((n, d)).astype(np.float32)
    grads = [(rng.standard_normal((n, d)) * 30.0 + 5.0 * np.sin(t + np.arange(n))[:, None]).astype(np.float32)
             for t in range(11)]
    zeros = np.zeros((n, d), np.float32)
    p = oracle_problem(m, K, eta, alpha, zeros, zeros, 0.0, 0)
    for v in _variants(n):
        # oracle trajectory in float64: state (x, y = gossiped tracker, g_new, g_old)
        ref = orc.State(x0.astype(np.float64), grads[0].astype(np.float64), grads[0].astype(np.float64),
                        grads[0].astype(np.float64), 0)
        with Session(m, d, K, eta, alpha, None, None, x0, variant=v, external_gradient=True) as s:
            assert B.detag_get_variant(s.state) == v
            s.upload("g_new", grads[0])
            s.init()
            assert np.array_equal(s.download("y"), grads[0]) and np.array_equal(s.download("g"), grads[0])
            for t in range(1, 11):
                # per element: one oracle step from the float32 state the GPU holds now (its own storage rounding)
                cur = orc.State(s.download("x").astype(np.float64), s.download("y").astype(np.float64),
                                grads[t].astype(np.float64), s.download("g").astype(np.float64), t - 1)
                y_f = orc.fold(cur.y, cur.g_new, cur.g_old)
                x_one, y_one = orc.gossip_and_update(p, cur.x, y_f)
                # the pure float64 trajectory
                yy = orc.fold(ref.y, grads[t].astype(np.float64), ref.g_old)
                xx, yy = orc.gossip_and_update(p, ref.x, yy)
                ref = orc.State(xx, yy, grads[t].astype(np.float64), grads[t].astype(np.float64), t)
                s.upload("g_new", grads[t])
                s.step()
                got_x, got_y, got_g = s.download("x"), s.download("y"), s.download("g")
                r = {"x": worst_ratio(got_x, x_one), "y": worst_ratio(got_y, y_one)}
                assert max(r.values()) <= 1.0, (v, t, r)
                assert np.array_equal(got_g, grads[t])  # the folded gradient is kept as the next g_old
                errs = {"x": rel_l2(got_x, ref.x), "y": rel_l2(got_y, ref.y)}
                assert max(errs.values()) <= 1e-4, (v, t, errs)
            s.status()


def test_external_gradient_misuse():
    import torch

    m = _graph("ring", 8)
    with Session(m, 64, 2, 0.2, 0.05, None, None, np.zeros((8, 64), np.float32), external_gradient=True) as s:
        with pytest.raises(B.DetagError) as e:
            s.step_many(2)  # one call per step: the caller has to supply each gradient
        assert e.value.code == B.DETAG_ERR_ARG
        with pytest.raises(B.DetagError) as e:
            B.detag_set_algorithm(s.state, B.DETAG_ALGORITHM_DPSGD)
        assert e.value.code == B.DETAG_ERR_UNSUPPORTED
        with pytest.raises(B.DetagError) as e:
            B.detag_set_gradient_source(s.state, B.DETAG_GRADIENT_EXTERNAL, s.g_new.data_ptr() + 4)
        assert e.value.code == B.DETAG_ERR_ARG
    # a state bound without objective data can step with caller-written gradients only
    st = B.detag_create(8, 64, m.row_ptr, m.col_idx, m.vals, 2, 0.2, 0.05)
    try:
        buf = torch.zeros((4, 8, 64), dtype=torch.float32, device="cuda:0")
        ws = torch.zeros(B.detag_workspace_bytes(st) + 256, dtype=torch.uint8, device="cuda:0")
        wsp = ws.data_ptr() + (-ws.data_ptr()) % 256
        B.detag_bind(st, 64, buf[0], buf[1], buf[2], None, None, wsp, ws.numel() - 256)
        for call in (B.detag_init, B.detag_step):
            with pytest.raises(B.DetagError) as e:
                call(st)
            assert e.value.code == B.DETAG_ERR_UNBOUND
        B.detag_set_gradient_source(st, B.DETAG_GRADIENT_EXTERNAL, buf[3])
        B.detag_init(st)
        B.detag_step(st)
        B.detag_status(st)
    finally:
        torch.cuda.synchronize()
        B.detag_destroy(st)
    m64 = _graph("ring", 64)
    with Session(m64, 64, 2, 0.2, 0.05, None, None, np.zeros((64, 64), np.float32), external_gradient=True) as s:
        B.detag_set_variant(s.state, B.DETAG_VARIANT_RING)  # the band kernel has no such mode
        with pytest.raises(B.DetagError) as e:
            s.step()
        assert e.value.code == B.DETAG_ERR_UNSUPPORTED
    torch.cuda.synchronize()


# ----------------------------------------------------------------------------- D-PSGD
def _objective(rng, n, d):
    a = rng.uniform(0.5, 2.0, (n, d)).astype(np.float32)
    c = (rng.standard_normal((n, d)) + np.arange(n)[:, None] - n / 2).astype(np.float32)
    return a, c


@pytest.mark.parametrize("n,d,K,eta_mode,kind", [(8, 300, 1, "zero", "ring"), (16, 1025, 1, "zero", "regular4"),
                                                  (32, 2050, 4, "spectral", "regular4"), (5, 37, 2, "spectral", "path"),
                                                  (6, 50, 1, "zero", "directed"), (40, 130, 1, "zero", "ring"),
                                                  (64, 67, 2, "spectral", "ring"), (128, 200, 1, "zero", "ring"),
                                                  (96, 64, 30, "spectral", "ring")])
def test_dpsgd_one_step_and_trajectory(n, d, K, eta_mode, kind):
    rng = np.random.default_rng(n * 17 + d)
    m = _graph(kind, n)
    eta = 0.0 if eta_mode == "zero" else orc.spectrum(m.to_dense()).eta
    a, c = _objective(rng, n, d)
    x0 = rng.standard_normal((n, d)).astype(np.float32)
    p = oracle_problem(m, K, eta, 0.05, a, c, 0.1, 13, 77)
    ref = []
    orc.run_dpsgd(p, x0, 8, observe=lambda st: ref.append((st.x.copy(), st.g.copy())))
    for v in _variants(n, dpsgd_ring=kind == "ring"):
        with Session(m, d, K, eta, 0.05, a, c, x0, 0.1, 13, coord_offset=77, variant=v,
                     algorithm=B.DETAG_ALGORITHM_DPSGD) as s:
            assert B.detag_get_algorithm(s.state) == B.DETAG_ALGORITHM_DPSGD
            s.y.fill_(4242.0)  # D-PSGD has no tracker: the buffer must stay untouched
            s.init()
            assert rel_l2(s.download("g"), ref[0][1]) <= 1e-6
            for t in range(1, 9):
                cur = orc.DpsgdState(s.download("x").astype(np.float64), s.download("g").astype(np.float64), t - 1)
                one = orc.dpsgd_step(p, cur)
                s.step()
                r = {"x": worst_ratio(s.download("x"), one.x), "g": worst_ratio(s.download("g"), one.g)}
                assert max(r.values()) <= 1.0, (v, t, r)
                errs = {"x": rel_l2(s.download("x"), ref[t][0]), "g": rel_l2(s.download("g"), ref[t][1])}
                assert max(errs.values()) <= 1e-4, (v, t, errs)
            s.status()
            assert bool((s.y == 4242.0).all())


def test_dpsgd_fused_call_and_host_resident_stepping_agree_with_single_steps():
    import torch

    rng = np.random.default_rng(99)
    n, d = 16, 20_003
    m = _graph("ring", n)
    a, c = _objective(rng, n, d)
    x0 = rng.standard_normal((n, d)).astype(np.float32)
    out = []
    for how in ("single", "many", "host"):
        with Session(m, d, 1, 0.0, 0.05, a, c, x0, 0.1, 3, algorithm=B.DETAG_ALGORITHM_DPSGD) as s:
            s.init()
            if how == "single":
                s.step(3)
            elif how == "many":
                s.step_many(3)
            else:
                host = {k: torch.empty((n, s.ld), dtype=torch.float32).pin_memory() for k in ("x", "y", "g", "a", "c")}
                for k in host:
                    host[k].copy_(getattr(s, k))
                torch.cuda.synchronize()
                nbytes = B.detag_host_staging_bytes(s.state, 4096)
                staging = torch.empty(nbytes + 256, dtype=torch.uint8, device="cuda:0")
                sptr = staging.data_ptr() + (-staging.data_ptr()) % 256
                for _ in range(3):
                    B.detag_step_host(s.state, s.ld, host["x"], host["y"], host["g"], host["a"], host["c"], sptr,
                                      nbytes, s.stream())
                torch.cuda.synchronize()
                s.status()
                out.append((host["x"][:, :d].numpy().copy(), host["g"][:, :d].numpy().copy()))
                continue
            s.status()
            out.append((s.download("x"), s.download("g")))
    for k in (1, 2):
        assert np.array_equal(out[0][0], out[k][0]) and np.array_equal(out[0][1], out[k][1])
