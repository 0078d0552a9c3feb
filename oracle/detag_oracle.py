"""Plain float64 CPU oracle of one DeTAG iteration over all n workers at once.

TEST INFRASTRUCTURE ONLY: used by tests, the smoke check and the benchmark's CPU-baseline
leg.  Shares no code with the CUDA path and never imports it.

Source of every formula: "Optimal Complexity in Decentralized Training" (arXiv 2006.08085).
Notation: the paper's phase length R (gossip rounds per phase) is called ``K`` here, one
phase is one *step*; ``M`` is the matrix applied row-wise, ``z'_i = sum_j M[i,j] z_j``,
i.e. ``M[i,j]`` is the paper's ``W_ji`` (Eq. "gossip update" and Algorithm 3).

State arrays have shape ``[n, m]``: worker i in row i, m coordinates (any coordinate
subset: the step never mixes coordinates).

Step (gradient evaluated last, at the new model; Algorithm 2 gives the updates):

    (a) fold      y   <- y + g_new - g_old                      Algorithm 2, tracker update
    (b) gossip    y   <- AG_K(y) ;  x <- AG_K(x) - alpha*y      Algorithm 2 (AG calls, model update)
    (c) gradient  g_old <- g_new ; g_new <- a*(x - c) + sigma*xi_t       stochastic oracle, Section "Setting"

with ``AG_K`` = Algorithm 3 and the initial state ``g_new = g_old = y = gradient(x0, t=0)``.

Noise.  ``xi`` is defined by a counter-based generator so that it is a pure function of
(seed, step t, worker i, coordinate j): Philox4x32-10 with key (seed low word, seed high word)
and counter (j low word, j high word, i // 4, t) yields four words r0..r3; the pair
(r0, r1) gives the normals of workers 4q and 4q+1, the pair (r2, r3) those of 4q+2 and
4q+3 (q = i // 4) by the Box-Muller transform with

    u_rad = ((r_even >> 9) + 0.5) * 2^-23   in (0, 1)
    u_ang = (r_odd >> 9) * 2^-23            in [0, 1)
    rad = sqrt(-2 ln u_rad) ;  first = rad*cos(2 pi u_ang) ;  second = rad*sin(2 pi u_ang).
"""
from __future__ import annotations

import math
from typing import NamedTuple, Optional, Tuple

import numpy as np

from .philox import philox4x32_10


# --------------------------------------------------------------------------------------
# Spectral quantities (Section "Protocol Layer"; Algorithm 3, momentum eta)
# --------------------------------------------------------------------------------------
class Spectrum(NamedTuple):
    lambda2: float  # second largest eigenvalue
    lambda_min: float  # smallest eigenvalue
    lam: float  # max(|lambda2|, |lambda_n|), the paper's lambda
    eta: float


def eta_from_lambda(lam: float) -> float:
    """Algorithm 3: eta = (1 - sqrt(1 - lambda^2)) / (1 + sqrt(1 - lambda^2))."""
    s = math.sqrt(1.0 - lam * lam)
    return (1.0 - s) / (1.0 + s)


def spectrum(w_dense: np.ndarray) -> Spectrum:
    """lambda = max(|lambda_2|, |lambda_n|) of a symmetric gossip matrix and the AG momentum."""
    w = np.asarray(w_dense, dtype=np.float64)
    if not np.allclose(w, w.T, atol=1e-12):
        raise ValueError("spectrum() needs a symmetric matrix")
    ev = np.linalg.eigvalsh(w)  # ascending
    lambda2 = float(ev[-2])
    lambda_min = float(ev[0])
    lam = max(abs(lambda2), abs(lambda_min))
    return Spectrum(lambda2, lambda_min, lam, eta_from_lambda(lam))


# --------------------------------------------------------------------------------------
# Accelerated gossip (Algorithm 3)
# --------------------------------------------------------------------------------------
def gossip_round(z: np.ndarray, row_ptr, col_idx, vals) -> np.ndarray:
    """One gossip step (Eq. "gossip update"): out_i = sum_j M[i,j] z_j over row i's entries."""
    z = np.asarray(z, dtype=np.float64)
    out = np.zeros_like(z)
    n = z.shape[0]
    for i in range(n):
        for k in range(int(row_ptr[i]), int(row_ptr[i + 1])):
            out[i] += float(vals[k]) * z[int(col_idx[k])]
    return out


def accelerated_gossip(z0: np.ndarray, row_ptr, col_idx, vals, K: int, eta: float) -> np.ndarray:
    """Algorithm 3 with R = K rounds: z_{-1} = z_0; z_{r+1} = (1+eta) M z_r - eta z_{r-1}."""
    z_prev = np.array(z0, dtype=np.float64, copy=True)
    z_cur = np.array(z0, dtype=np.float64, copy=True)
    for _ in range(K):
        z_next = (1.0 + eta) * gossip_round(z_cur, row_ptr, col_idx, vals) - eta * z_prev
        z_prev, z_cur = z_cur, z_next
    return z_cur


# --------------------------------------------------------------------------------------
# Stochastic gradient of the synthetic objective
# --------------------------------------------------------------------------------------
def standard_normal_noise(seed: int, t: int, n: int, j0: int, j1: int) -> np.ndarray:
    """xi[i, j-j0] for workers 0..n-1 and coordinates j0 <= j < j1 at step t (see module docstring)."""
    m = j1 - j0
    j = np.arange(j0, j1, dtype=np.uint64)
    nq = (n + 3) // 4
    q = np.arange(nq, dtype=np.uint64)
    r = philox4x32_10(j[None, :] & np.uint64(0xFFFFFFFF), j[None, :] >> np.uint64(32), q[:, None],
                      np.uint64(t), seed & 0xFFFFFFFF, (seed >> 32) & 0xFFFFFFFF)
    out = np.empty((nq * 4, m), dtype=np.float64)
    for p in range(2):
        u_rad = ((r[2 * p] >> np.uint32(9)).astype(np.float64) + 0.5) * 2.0 ** -23
        u_ang = (r[2 * p + 1] >> np.uint32(9)).astype(np.float64) * 2.0 ** -23
        rad = np.sqrt(-2.0 * np.log(u_rad))
        out[2 * p::4] = rad * np.cos(2.0 * math.pi * u_ang)
        out[2 * p + 1::4] = rad * np.sin(2.0 * math.pi * u_ang)
    return out[:n]


def gradient(x: np.ndarray, a: np.ndarray, c: np.ndarray, sigma: float, xi: Optional[np.ndarray]) -> np.ndarray:
    """g_i = a_i * (x_i - c_i) + sigma * xi_i: exact gradient of 1/2 sum_j a_ij (x_j - c_ij)^2 plus noise."""
    g = np.asarray(a, dtype=np.float64) * (np.asarray(x, dtype=np.float64) - np.asarray(c, dtype=np.float64))
    if xi is not None and sigma != 0.0:
        g = g + sigma * xi
    return g


# --------------------------------------------------------------------------------------
# The DeTAG step
# --------------------------------------------------------------------------------------
class Problem(NamedTuple):
    """Everything that stays fixed over a run, for one coordinate range [j0, j0+m)."""
    row_ptr: np.ndarray
    col_idx: np.ndarray
    vals: np.ndarray  # entries of M (row-applied matrix, M[i,j] = W_ji)
    K: int
    eta: float
    alpha: float
    a: np.ndarray  # [n, m]
    c: np.ndarray  # [n, m]
    sigma: float
    seed: int
    j0: int = 0  # global index of column 0 (enters the noise counter)


class State(NamedTuple):
    x: np.ndarray
    y: np.ndarray  # tracker after the gossip of the last step (or y0)
    g_new: np.ndarray  # stochastic gradient at the current x
    g_old: np.ndarray  # the one before
    t: int  # number of completed steps


def stochastic_gradient(p: Problem, x: np.ndarray, t: int) -> np.ndarray:
    n, m = x.shape
    xi = standard_normal_noise(p.seed, t, n, p.j0, p.j0 + m) if p.sigma != 0.0 else None
    return gradient(x, p.a, p.c, p.sigma, xi)


def init_state(p: Problem, x0: np.ndarray) -> State:
    """y0 = g(x0); both gradient buffers hold g(x0), so the first fold changes nothing."""
    x = np.array(x0, dtype=np.float64, copy=True)
    g = stochastic_gradient(p, x, 0)
    return State(x, g.copy(), g, g.copy(), 0)


def fold(y: np.ndarray, g_new: np.ndarray, g_old: np.ndarray) -> np.ndarray:
    """(a) tracker update of Algorithm 2: y + g_(k) - g_(k-1)."""
    return np.asarray(y, dtype=np.float64) + np.asarray(g_new, dtype=np.float64) - np.asarray(g_old, dtype=np.float64)


def gossip_and_update(p: Problem, x: np.ndarray, y_folded: np.ndarray) -> Tuple[np.ndarray, np.ndarray]:
    """(b): accelerated gossip on tracker and model, then x <- x~ - alpha*y with the gossiped tracker."""
    y = accelerated_gossip(y_folded, p.row_ptr, p.col_idx, p.vals, p.K, p.eta)
    x_tilde = accelerated_gossip(x, p.row_ptr, p.col_idx, p.vals, p.K, p.eta)
    return x_tilde - p.alpha * y, y


def step(p: Problem, s: State) -> State:
    """One DeTAG iteration: (a) fold, (b) gossip + model update, (c) new stochastic gradient."""
    y = fold(s.y, s.g_new, s.g_old)
    x, y = gossip_and_update(p, s.x, y)
    g = stochastic_gradient(p, x, s.t + 1)
    return State(x, y, g, s.g_new, s.t + 1)


def folded_tracker(s: State) -> np.ndarray:
    """The tracker as the next step's (a) will see it: y + g_new - g_old."""
    return fold(s.y, s.g_new, s.g_old)


# --------------------------------------------------------------------------------------
# Algorithm 2 with the timing it prints: the gradient of phase k is queried at the phase-start point
# --------------------------------------------------------------------------------------
class PhaseState(NamedTuple):
    """State at the start of phase k of Algorithm 2 read literally."""
    x: np.ndarray  # x_k
    y: np.ndarray  # tracker y_k as the algorithm holds it (the fold of phase k-1 already applied)
    g_prev: np.ndarray  # gradient buffer g_(k-1)
    t: int  # number of completed phases


def init_phase_state(p: Problem, x0: np.ndarray) -> PhaseState:
    """Same start as ``init_state``: y_0 = g_(-1) = stochastic gradient at x_0 (noise index 0)."""
    x = np.array(x0, dtype=np.float64, copy=True)
    g = stochastic_gradient(p, x, 0)
    return PhaseState(x, g.copy(), g, 0)


def phase_as_printed(p: Problem, s: PhaseState) -> PhaseState:
    """One phase of Algorithm 2 in the order the algorithm box prints it.

    While the K gossip rounds run on the model replica and on the tracker, the gradient oracle is
    queried at the phase-start point x_k (the box's "compute stochastic gradient at point x_k");
    at the end of the phase the model is updated with the gossiped tracker and only then is the
    tracker folded with g_(k) - g_(k-1).  Compared with ``step`` the gradient that enters a fold
    is one phase older.
    """
    g = stochastic_gradient(p, s.x, s.t + 1)
    y_gossip = accelerated_gossip(s.y, p.row_ptr, p.col_idx, p.vals, p.K, p.eta)
    x_tilde = accelerated_gossip(s.x, p.row_ptr, p.col_idx, p.vals, p.K, p.eta)
    x = x_tilde - p.alpha * y_gossip
    y = y_gossip + g - s.g_prev
    return PhaseState(x, y, g, s.t + 1)


def run_as_printed(p: Problem, x0: np.ndarray, phases: int, observe=None) -> PhaseState:
    s = init_phase_state(p, x0)
    if observe is not None:
        observe(s)
    for _ in range(phases):
        s = phase_as_printed(p, s)
        if observe is not None:
            observe(s)
    return s


# --------------------------------------------------------------------------------------
# D-PSGD, the paper's main baseline (Section "Related work"; baselines of Section "Experiments")
# --------------------------------------------------------------------------------------
class DpsgdState(NamedTuple):
    x: np.ndarray
    g: np.ndarray  # stochastic gradient at the current x
    t: int  # number of completed steps


def init_dpsgd_state(p: Problem, x0: np.ndarray) -> DpsgdState:
    x = np.array(x0, dtype=np.float64, copy=True)
    return DpsgdState(x, stochastic_gradient(p, x, 0), 0)


def dpsgd_step(p: Problem, s: DpsgdState) -> DpsgdState:
    """Every worker averages its neighbours' models with the gossip matrix and steps along its own stochastic
    gradient taken at its own current model: x' = AG_K(x) - alpha * g(x).  Plain D-PSGD is K = 1, eta = 0, where
    AG_K is one gossip step, x'_i = sum_j W_ji x_j - alpha g_i.  No tracker."""
    x = accelerated_gossip(s.x, p.row_ptr, p.col_idx, p.vals, p.K, p.eta) - p.alpha * s.g
    return DpsgdState(x, stochastic_gradient(p, x, s.t + 1), s.t + 1)


def run_dpsgd(p: Problem, x0: np.ndarray, steps: int, observe=None) -> DpsgdState:
    s = init_dpsgd_state(p, x0)
    if observe is not None:
        observe(s)
    for _ in range(steps):
        s = dpsgd_step(p, s)
        if observe is not None:
            observe(s)
    return s


def phase_length(n: int, lam: float, varsigma0_sq: float, T: float, delta_L: float) -> int:
    """Theorem 3's phase length R = max(1/2 ln n, 1/2 ln(varsigma_0^2 T / (Delta L))) / sqrt(1 - lambda),
    rounded up to a whole number of gossip rounds (at least one)."""
    terms = [0.5 * math.log(n)]
    if varsigma0_sq > 0.0 and T > 0.0 and delta_L > 0.0:
        terms.append(0.5 * math.log(varsigma0_sq * T / delta_L))
    return max(1, math.ceil(max(terms) / math.sqrt(1.0 - lam)))


def consensus_error(x: np.ndarray) -> float:
    """||X - Xbar 1^T||_F^2 = sum_j sum_i (x_ij - mean_i x_ij)^2."""
    x = np.asarray(x, dtype=np.float64)
    return float(((x - x.mean(axis=0, keepdims=True)) ** 2).sum())


def run(p: Problem, x0: np.ndarray, steps: int, observe=None) -> State:
    """init + `steps` iterations; ``observe(state)`` is called after init and after every step."""
    s = init_state(p, x0)
    if observe is not None:
        observe(s)
    for _ in range(steps):
        s = step(p, s)
        if observe is not None:
            observe(s)
    return s
