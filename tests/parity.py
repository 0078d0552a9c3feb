"""Shared pieces of the GPU-vs-oracle parity tests (tolerances, oracle problem assembly)."""
import numpy as np

from oracle import detag_oracle as orc


def oracle_problem(m, K, eta, alpha, a, c, sigma, seed, j0=0):
    return orc.Problem(m.row_ptr, m.col_idx, m.vals, K, eta, alpha, a, c, sigma, seed, j0)


def worst_ratio(got, ref, extra=None):
    """max |got-ref| / (1e-5 (1+|ref|) [+ extra]) : the per-element bound holds iff this is <= 1."""
    tol = 1e-5 * (1.0 + np.abs(ref))
    if extra is not None:
        tol = tol + extra
    return float((np.abs(got.astype(np.float64) - ref) / tol).max()) if ref.size else 0.0


def rel_l2(got, ref):
    den = float(np.sqrt((ref ** 2).sum()))
    num = float(np.sqrt(((got.astype(np.float64) - ref) ** 2).sum()))
    return num / den if den > 0 else num


def one_step_from_rounded_state(p, x0):
    """Oracle: init in float64, round the state to the float32 storage type, then one step from it.

    Returns the float32 start state (x, y, g) and the float64 results after the step in the library's
    storage convention: x', gossiped tracker y~, g', folded tracker y' = y~ + g' - g.
    """
    s0 = orc.init_state(p, x0)
    x32, y32, g32 = (v.astype(np.float32) for v in (s0.x, s0.y, s0.g_new))
    x_new, y_gossip = orc.gossip_and_update(p, x32, y32)  # the first fold is the identity (g_new == g_old)
    g_new = orc.stochastic_gradient(p, x_new, 1)
    y_fold = orc.fold(y_gossip, g_new, g32)
    return (x32, y32, g32), (x_new, y_gossip, g_new, y_fold)


HALF_ULP32 = 2.0 ** -24  # the stored float32 gradient the tracker telescopes against is off by <= this (relative)
