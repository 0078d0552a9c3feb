"""The scratch-free consensus-error entry point (collected last on purpose: see the file name).

`detag_consensus_error_static` serves callers that can neither allocate device memory nor hand the
library a workspace (a hook running where cudaMalloc is off limits, a plug-in that only sees the model
buffer).  It must agree with the ordinary `detag_consensus_error`, which works out of the caller's
workspace, and it must keep doing so when called repeatedly: all calls share one array built into the
library, and that array still holds whatever the previous call left there.
"""
import numpy as np
import pytest

from oracle import detag_oracle as orc
from paper_2006_08085_b200 import binding as B
from paper_2006_08085_b200 import build, inputs
from paper_2006_08085_b200.session import Session

pytestmark = pytest.mark.gpu


def test_static_scratch_consensus_error_matches_the_workspace_one_twice_in_a_row():
    build.build()
    rng = np.random.default_rng(2024)
    n, d = 16, 300_007  # many 256-coordinate blocks and a ragged last one
    m = inputs.metropolis_weights(inputs.ring_graph(n))
    ones = np.ones((n, d), dtype=np.float32)
    x_first = (rng.standard_normal((n, d)) * 2.0 + 10.0).astype(np.float32)
    # second call: fewer coordinates and other values, so stale partial sums of the first call sit
    # right behind the slots the second call uses
    d_second = 70_001
    x_second = (rng.standard_normal((n, d_second)) * 0.5 - 3.0).astype(np.float32)
    with Session(m, d, 2, 0.1, 0.1, ones, ones, x_first) as s1, \
            Session(m, d_second, 2, 0.1, 0.1, ones[:, :d_second], ones[:, :d_second], x_second) as s2:
        for s, dd, host in ((s1, d, x_first), (s2, d_second, x_second), (s1, d, x_first)):
            want = B.detag_consensus_error(s.state, s.stream())
            got = B.detag_consensus_error_static(n, dd, s.ld, s.x, s.stream())
            assert want > 0.0
            assert got == pytest.approx(want, rel=1e-12)
            # and against the definition, evaluated by the CPU oracle on the same float32 array
            assert got == pytest.approx(orc.consensus_error(host), rel=1e-12)
        # beyond the built-in array: refused, nothing launched
        with pytest.raises(B.DetagError) as e:
            B.detag_consensus_error_static(n, 33_554_432 + 1, 33_554_436, s1.x, s1.stream())
        assert e.value.code == B.DETAG_ERR_UNSUPPORTED
        # arguments that make no sense are refused as such
        for args in ((n, d, d - 4, s1.x), (0, d, s1.ld, s1.x), (n, 0, s1.ld, s1.x), (n, d, s1.ld, None)):
            with pytest.raises(B.DetagError) as e:
                B.detag_consensus_error_static(*args, s1.stream())
            assert e.value.code == B.DETAG_ERR_ARG


def test_static_scratch_at_its_size_limit():
    """Exactly the largest supported size: the last slot of the built-in array and the result slot behind it are
    in use.  Two workers keep the caller's own array at 268 MB; the library still allocates nothing."""
    import torch

    build.build()
    n, d = 2, 33_554_432
    m = inputs.metropolis_weights(inputs.complete_graph(2))
    g = torch.Generator(device="cuda:0").manual_seed(5)
    x = torch.randn((n, d), dtype=torch.float32, device="cuda:0", generator=g)
    x[0, -3:] += 1000.0  # the very last block must count
    got = B.detag_consensus_error_static(n, d, d, x, None)
    # definition in float64 on the same values: sum_j (x_0j - x_1j)^2 / 2 for two workers
    want = float(((x[0].double() - x[1].double()) ** 2).sum().item() / 2.0)
    assert got == pytest.approx(want, rel=1e-10)
    st = B.detag_create(n, d, m.row_ptr, m.col_idx, m.vals, 1, 0.0, 0.1)
    try:
        ws = torch.zeros(B.detag_workspace_bytes(st) + 256, dtype=torch.uint8, device="cuda:0")
        wsp = ws.data_ptr() + (-ws.data_ptr()) % 256
        B.detag_bind(st, d, x, x, x, x, x, wsp, ws.numel() - 256)
        assert got == pytest.approx(B.detag_consensus_error(st), rel=1e-12)
    finally:
        B.detag_destroy(st)
