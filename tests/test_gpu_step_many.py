"""detag_step_many: several iterations per call.  Where the fused on-chip kernel applies (dense polynomial, n <= 32)
its results must be bit-identical to the same number of detag_step calls; elsewhere the call is that loop."""
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


def _case(n, d, seed):
    rng = np.random.default_rng(seed)
    m = inputs.metropolis_weights(inputs.ring_graph(n))
    eta = orc.spectrum(m.to_dense()).eta
    a = rng.uniform(0.5, 2.0, (n, d)).astype(np.float32)
    c = (rng.standard_normal((n, d)) + np.arange(n)[:, None] - n / 2).astype(np.float32)
    x0 = rng.standard_normal((n, d)).astype(np.float32)
    return m, eta, a, c, x0


@pytest.mark.parametrize("n,d,K,count", [(8, 4096, 2, 10), (16, 10_003, 4, 7), (32, 20_001, 6, 5), (5, 37, 3, 4), (3, 2, 1, 3),
                                         (8, 64, 2, 1030)])  # more than one launch's worth of fused steps
@pytest.mark.parametrize("where", [B.DETAG_GRADIENT_AT_NEW_MODEL, B.DETAG_GRADIENT_AT_PHASE_START])
def test_fused_steps_equal_single_steps_bit_for_bit(n, d, K, count, where):
    m, eta, a, c, x0 = _case(n, d, n + d)
    got = []
    for fused in (False, True):
        with Session(m, d, K, eta, 0.05, a, c, x0, 0.1, 9, coord_offset=123, gradient_point=where) as s:
            assert B.detag_get_variant(s.state) == B.DETAG_VARIANT_DENSE
            s.init()
            if fused:
                s.step_many(count)
                s.step_many(2)  # a second call continues from the step counter
            else:
                s.step(count + 2)
            s.status()
            assert B.detag_get_step(s.state) == count + 2
            got.append({k: s.download(k) for k in ("x", "y", "g")})
    for k in ("x", "y", "g"):
        assert np.array_equal(got[0][k], got[1][k]), k


def test_fused_trajectory_against_the_oracle():
    n, d, K, steps = 16, 3_001, 4, 12
    m, eta, a, c, x0 = _case(n, d, 5)
    p = oracle_problem(m, K, eta, 0.05, a, c, 0.1, 4)
    ref = orc.run(p, x0, steps)
    with Session(m, d, K, eta, 0.05, a, c, x0, 0.1, 4) as s:
        s.init()
        s.step_many(steps)
        s.status()
        for k, want in (("x", ref.x), ("y", orc.folded_tracker(ref)), ("g", ref.g_new)):
            assert rel_l2(s.download(k), want) <= 1e-4, k


def test_other_variants_loop_over_single_steps():
    """n = 64 (no fused kernel) and a forced CSR variant: the call is `count` single steps."""
    for n, variant in ((64, B.DETAG_VARIANT_AUTO), (8, B.DETAG_VARIANT_CSR)):
        m, eta, a, c, x0 = _case(n, 700, n)
        got = []
        for many in (False, True):
            with Session(m, 700, 3, eta, 0.02, a, c, x0, 0.1, 2, variant=variant) as s:
                s.init()
                s.step_many(4) if many else s.step(4)
                s.status()
                got.append(s.download("y"))
        assert np.array_equal(got[0], got[1])


def test_count_must_be_positive():
    m, eta, a, c, x0 = _case(4, 16, 1)
    with Session(m, 16, 2, eta, 0.05, a, c, x0) as s:
        with pytest.raises(B.DetagError) as e:
            s.step_many(0)
        assert e.value.code == B.DETAG_ERR_ARG
