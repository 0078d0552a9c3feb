"""Failure detection on the GPU without a fault: bounded device-side waits that run out.

Every wait in the kernels (mbarrier phases, progress counters) is bounded by a poll limit; a wait that gives up
sets a status word, the waiting role winds down and the launch ends normally.  Here the limit is made small and
the failure is made on purpose - a barrier nobody arrives at, or a loading thread that stops loading - and the
host must see DETAG_ERR_TIMEOUT, the context must stay usable, and a re-bound state must step correctly again.
Nothing in these tests traps, faults or waits without a limit.
"""
import numpy as np
import pytest

from oracle import detag_oracle as orc
from paper_2006_08085_b200 import binding as B
from paper_2006_08085_b200 import build, inputs
from paper_2006_08085_b200.session import Session
from parity import oracle_problem, rel_l2

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _built():
    build.build()


def _case(n, d, seed=0, torus=False):
    rng = np.random.default_rng(seed)
    m = inputs.metropolis_weights(inputs.torus_graph(n // 8, 8) if torus else inputs.ring_graph(n))
    a = rng.uniform(0.5, 2.0, (n, d)).astype(np.float32)
    c = rng.standard_normal((n, d)).astype(np.float32)
    x0 = rng.standard_normal((n, d)).astype(np.float32)
    return m, a, c, x0


def _rebind(s):
    B.detag_bind(s.state, s.ld, s.x, s.y, s.g, s.a, s.c, s._ws_ptr, s._ws_bytes)  # clears the status word


def test_a_wait_that_nothing_ends_gives_up_and_is_reported():
    m, a, c, x0 = _case(8, 256)
    with Session(m, 256, 2, 0.2, 0.05, a, c, x0) as s:
        s.init()
        s.status()
        B.detag_debug_expire_wait(s.state, 3000, s.stream())
        with pytest.raises(B.DetagError) as e:
            s.status()
        assert e.value.code == B.DETAG_ERR_TIMEOUT
        with pytest.raises(B.DetagError):  # the word is sticky until the workspace is bound again
            s.status()
        _rebind(s)
        s.status()
        s.step(2)  # the context is intact: kernels still run
        s.status()


@pytest.mark.parametrize("n,d,K,variant,after", [
    (16, 64 * 148 * 4 + 17, 3, B.DETAG_VARIANT_DENSE, 1),   # dense kernel, n <= 32: several slabs per CTA
    (16, 64 * 148 * 4 + 17, 3, B.DETAG_VARIANT_DENSE, 0),   # nothing is ever loaded
    (64, 64 * 148 * 2 + 5, 2, B.DETAG_VARIANT_RING, 3),     # band kernel, ring
    (48, 64 * 148 * 2 + 5, 2, B.DETAG_VARIANT_DENSE, 1),    # band kernel, dense window mode
    (64, 64 * 148 * 3 + 5, 2, B.DETAG_VARIANT_TORUS, 2),    # block-circulant transform kernel
    (32, 64 * 148 * 3 + 5, 2, B.DETAG_VARIANT_TORUS, 0),
    (72, 64 * 148 * 2 + 5, 2, B.DETAG_VARIANT_DENSE, 1),    # dense kernel with the polynomial in registers, two stages of g, a, c
    (128, 64 * 148 * 2 + 37, 2, B.DETAG_VARIANT_DENSE, 0),  # ... one stage
])
def test_a_stalled_loader_times_out_every_waiter_and_the_state_recovers(n, d, K, variant, after):
    m, a, c, x0 = _case(n, d, n, torus=variant == B.DETAG_VARIANT_TORUS)
    eta = orc.spectrum(m.to_dense()).eta
    p = oracle_problem(m, K, eta, 0.05, a, c, 0.1, 7)
    ref = orc.run(p, x0, 2)
    with Session(m, d, K, eta, 0.05, a, c, x0, 0.1, 7, variant=variant) as s:
        s.init()
        B.detag_debug_inject_stall(s.state, after, 2048)
        s.step()  # the launch itself succeeds; its CTAs give up one wait after the other and return
        with pytest.raises(B.DetagError) as e:
            s.status()
        assert e.value.code == B.DETAG_ERR_TIMEOUT and "wait gave up" in B.detag_last_error(s.state)
        # recovery: normal operation again, fresh state, correct results
        B.detag_debug_inject_stall(s.state, -1, 0)
        _rebind(s)
        s.upload("x", x0)
        s.init()
        s.step(2)
        s.status()
        assert rel_l2(s.download("x"), ref.x) <= 1e-4
        assert rel_l2(s.download("y"), orc.folded_tracker(ref)) <= 1e-4


def test_status_after_host_resident_stepping_needs_no_bind_and_sees_a_timeout():
    import torch

    n, d = 16, 40_000
    m, a, c, x0 = _case(n, d, 3)
    st = B.detag_create(n, d, m.row_ptr, m.col_idx, m.vals, 2, 0.2, 0.05)
    try:
        with pytest.raises(B.DetagError) as e:
            B.detag_status(st)  # neither bound nor stepped
        assert e.value.code == B.DETAG_ERR_UNBOUND
        host = {k: torch.zeros((n, d), dtype=torch.float32).pin_memory() for k in ("x", "y", "g", "a", "c")}
        host["a"].copy_(torch.from_numpy(a))
        host["c"].copy_(torch.from_numpy(c))
        host["x"].copy_(torch.from_numpy(x0))
        nbytes = B.detag_host_staging_bytes(st, 8192)
        staging = torch.empty(nbytes + 256, dtype=torch.uint8, device="cuda:0")
        sptr = staging.data_ptr() + (-staging.data_ptr()) % 256
        args = (st, d, host["x"], host["y"], host["g"], host["a"], host["c"], sptr, nbytes)
        B.detag_step_host(*args)
        B.detag_status(st)  # a state that was never bound: reads the staging area's word
        B.detag_debug_inject_stall(st, 0, 2048)
        B.detag_step_host(*args)
        with pytest.raises(B.DetagError) as e:
            B.detag_status(st)
        assert e.value.code == B.DETAG_ERR_TIMEOUT
        B.detag_debug_inject_stall(st, -1, 0)
        B.detag_step_host(*args)  # same staging area: the word is not cleared behind the caller's back
        with pytest.raises(B.DetagError) as e:
            B.detag_status(st)
        assert e.value.code == B.DETAG_ERR_TIMEOUT
        torch.cuda.synchronize()
    finally:
        B.detag_destroy(st)


def test_injection_arguments_are_checked():
    m, a, c, x0 = _case(4, 16)
    st = B.detag_create(4, 16, m.row_ptr, m.col_idx, m.vals, 2, 0.1, 0.1)
    try:
        for after, polls in ((0, 0), (0, 15), (1, (1 << 20) + 1)):
            with pytest.raises(B.DetagError) as e:
                B.detag_debug_inject_stall(st, after, polls)
            assert e.value.code == B.DETAG_ERR_ARG
        with pytest.raises(B.DetagError) as e:
            B.detag_debug_expire_wait(st, 100)
        assert e.value.code == B.DETAG_ERR_UNBOUND
    finally:
        B.detag_destroy(st)
