"""The zero-chain objective of the paper's lower-bound construction (proof of Theorem 1) on the GPU: its gradient
oracle against the float64 oracle per element, and DeTAG driven by it through caller-written gradients against the
oracle's trajectory (complete graph, as in the proof's first setting)."""
import numpy as np
import pytest

from oracle import detag_oracle as orc
from oracle import zero_chain as zc
from paper_2006_08085_b200 import binding as B
from paper_2006_08085_b200 import build, inputs
from paper_2006_08085_b200.session import Session
from parity import oracle_problem, rel_l2, worst_ratio

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _built():
    build.build()


@pytest.mark.parametrize("n,d,ld,p", [(4, 16, 16, 1.0), (7, 1000, 1004, 0.3), (16, 4097, 4100, 0.05), (3, 1, 4, 0.5)])
def test_gradient_oracle_per_element(n, d, ld, p):
    import torch

    rng = np.random.default_rng(n + d)
    x = np.zeros((n, d), dtype=np.float32)
    for i in range(n):  # different progress per worker, values on both sides of the kinks of Psi
        k = int(rng.integers(0, d + 1))
        x[i, :k] = rng.uniform(-1.5, 1.5, k)
    xt = torch.zeros((n, ld), dtype=torch.float32, device="cuda:0")
    xt[:, :d] = torch.from_numpy(x)
    g = torch.full((n, ld), 777.0, dtype=torch.float32, device="cuda:0")
    scratch = torch.empty(n, dtype=torch.int32, device="cuda:0")
    lam, gain = 0.7, 2.5
    for t in (0, 3):
        B.detag_zero_chain_gradient(n, d, ld, xt, g, lam, gain, p, 99, t, scratch)
        torch.cuda.synchronize()
        want = zc.stochastic_gradient(x, lam, gain, p, 99, t)
        assert worst_ratio(g[:, :d].cpu().numpy(), want) <= 1.0
        assert np.array_equal(scratch.cpu().numpy(), zc.prog(x))
        assert bool((g[:, d:] == 777.0).all())  # padding untouched
    for bad in ((n, d, d - 1 if d > 1 else 0, xt, g, lam, gain, p), (n, d, ld, xt, g, 0.0, gain, p), (n, d, ld, xt, g, lam, gain, 0.0),
                (n, d, ld, xt, g, lam, gain, 1.5), (n, d, ld, None, g, lam, gain, p)):
        with pytest.raises(B.DetagError) as e:
            B.detag_zero_chain_gradient(*bad, 1, 0, scratch)
        assert e.value.code == B.DETAG_ERR_ARG


def test_detag_on_the_zero_chain_through_caller_written_gradients():
    """n workers on the complete graph (uniform weights), every worker holding the rescaled chain; DeTAG advances
    along the chain one coordinate per successful draw.  GPU (gradient kernel + step with caller-written
    gradients) against the float64 oracle, same Bernoulli draws on both sides."""
    n, T, K, steps = 8, 48, 2, 150
    # f = (L lam^2 / l_1) fhat(x / lam) with L = 20 (l_1 = 152 is fhat's smoothness); alpha L = 0.8
    lam, p, alpha, seed = 0.5, 0.5, 0.04, 7
    gain = 20.0 * lam / 152.0
    m = inputs.average_consensus_matrix(n)
    zeros = np.zeros((n, T), np.float32)
    prob = oracle_problem(m, K, 0.0, alpha, zeros, zeros, 0.0, 0)
    g0 = zc.stochastic_gradient(zeros, lam, gain, p, seed, 0)
    ref = orc.State(zeros.astype(np.float64), g0.copy(), g0.copy(), g0.copy(), 0)
    with Session(m, T, K, 0.0, alpha, None, None, zeros, external_gradient=True) as s:
        import torch
        scratch = torch.empty(n, dtype=torch.int32, device="cuda:0")
        B.detag_zero_chain_gradient(n, T, s.ld, s.x, s.g_new, lam, gain, p, seed, 0, scratch, s.stream())
        s.init()
        reached = 0
        for t in range(1, steps + 1):
            # oracle: fold + gossip + update with the gradient evaluated at the model the step starts from
            y = orc.fold(ref.y, ref.g_new, ref.g_old)
            x, y = orc.gossip_and_update(prob, ref.x, y)
            g = zc.stochastic_gradient(x, lam, gain, p, seed, t)
            ref = orc.State(x, y, g, ref.g_new, t)
            s.step()
            B.detag_zero_chain_gradient(n, T, s.ld, s.x, s.g_new, lam, gain, p, seed, t, scratch, s.stream())
            assert rel_l2(s.download("x"), ref.x) <= 1e-4 and rel_l2(s.download("y"), ref.y) <= 1e-4, t
            assert rel_l2(s.download("g_new"), ref.g_new) <= 1e-4, t
            reached = int(zc.prog(s.download("x")).max())
        s.status()
        assert 2 <= reached <= steps + 1  # the chain is being climbed, at most one coordinate per step
