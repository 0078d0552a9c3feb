"""Seeded synthetic inputs for the DeTAG step: graphs, gossip matrices, objective data.

This module only *draws inputs*.  It holds none of the method's arithmetic (no gossip,
no tracker, no gradient, no noise transform): the CPU oracle and the CUDA library each
implement those on their own and are both fed from here.

Gossip matrices follow the paper's setting (Section "Protocol Layer"): doubly stochastic,
non-zero only on the graph's edges and the diagonal.  Rings use Metropolis weights, as in
the paper's second experiment, and the slack family ``W_kappa = kappa*W0 + (1-kappa)*I``
is available for the small-spectral-gap regime.

Objective data.  Worker ``i`` holds ``f_i(x) = 1/2 * sum_j a_ij (x_j - c_ij)^2``.  The arrays
``a`` and ``c`` (shape ``[n, d]``) and the start point ``x0`` are drawn in float64 and rounded
once to float32; both consumers receive those float32 values.

Random access.  Every array is drawn in independent blocks of ``BLOCK`` coordinates, one
numpy ``Philox`` stream per (seed, array, worker, block), so any coordinate range of a
25.6M-wide config can be produced without drawing the rest.
"""
from __future__ import annotations

import math
from concurrent.futures import ThreadPoolExecutor
from dataclasses import dataclass, field
from typing import Callable, Dict, List, Optional, Sequence, Tuple

import numpy as np

BLOCK = 1 << 16  # coordinates per independently seeded block

# stream ids of the per-config arrays
_STREAM_A, _STREAM_C, _STREAM_X0, _STREAM_MU, _STREAM_GRAPH = 1, 2, 3, 4, 5


# --------------------------------------------------------------------------------------
# Sparse matrices
# --------------------------------------------------------------------------------------
@dataclass(frozen=True)
class CSR:
    """Row-compressed n x n matrix; columns sorted within each row.

    ``vals[k]`` with ``row_ptr[i] <= k < row_ptr[i+1]`` is the entry (i, col_idx[k]).
    """

    n: int
    row_ptr: np.ndarray  # int32 [n+1]
    col_idx: np.ndarray  # int32 [nnz]
    vals: np.ndarray  # float64 [nnz]

    @property
    def nnz(self) -> int:
        return int(self.col_idx.shape[0])

    def to_dense(self) -> np.ndarray:
        m = np.zeros((self.n, self.n), dtype=np.float64)
        for i in range(self.n):
            for k in range(self.row_ptr[i], self.row_ptr[i + 1]):
                m[i, self.col_idx[k]] += self.vals[k]
        return m

    def transposed(self) -> "CSR":
        t = self.to_dense().T
        return csr_from_dense(t, keep=t != 0)


def csr_from_dense(m: np.ndarray, keep: Optional[np.ndarray] = None) -> CSR:
    m = np.asarray(m, dtype=np.float64)
    n = m.shape[0]
    if keep is None:
        keep = m != 0
    row_ptr = np.zeros(n + 1, dtype=np.int32)
    cols: List[int] = []
    vals: List[float] = []
    for i in range(n):
        js = np.nonzero(keep[i])[0]
        cols.extend(int(j) for j in js)
        vals.extend(float(m[i, j]) for j in js)
        row_ptr[i + 1] = len(cols)
    return CSR(n, row_ptr, np.asarray(cols, dtype=np.int32), np.asarray(vals, dtype=np.float64))


# --------------------------------------------------------------------------------------
# Graphs (undirected, as sorted neighbour lists without self loops)
# --------------------------------------------------------------------------------------
Adjacency = List[List[int]]


def ring_graph(n: int) -> Adjacency:
    if n < 3:
        raise ValueError("a ring needs n >= 3")
    return [sorted({(i - 1) % n, (i + 1) % n}) for i in range(n)]


def path_graph(n: int) -> Adjacency:
    return [[j for j in (i - 1, i + 1) if 0 <= j < n] for i in range(n)]


def complete_graph(n: int) -> Adjacency:
    return [[j for j in range(n) if j != i] for i in range(n)]


def torus_graph(rows: int, cols: int) -> Adjacency:
    """rows x cols grid with wrap-around; vertex (r, c) has index r*cols + c."""
    if rows < 3 or cols < 3:
        raise ValueError("torus sides must be >= 3 so the four neighbours are distinct")
    adj: Adjacency = []
    for r in range(rows):
        for c in range(cols):
            nb = {((r - 1) % rows) * cols + c, ((r + 1) % rows) * cols + c,
                  r * cols + (c - 1) % cols, r * cols + (c + 1) % cols}
            adj.append(sorted(nb))
    return adj


def random_regular4_graph(n: int, seed: int) -> Adjacency:
    """Seeded connected 4-regular graph: the union of two random Hamiltonian cycles.

    The second cycle is redrawn until it shares no edge with the first, so every vertex
    has exactly four distinct neighbours; a Hamiltonian cycle makes the graph connected.
    """
    if n < 5:
        raise ValueError("need n >= 5 for two edge-disjoint Hamiltonian cycles")
    rng = np.random.Generator(np.random.Philox(key=[np.uint64(seed), np.uint64(_STREAM_GRAPH << 48)]))

    def cycle_edges(perm: np.ndarray) -> set:
        return {frozenset((int(perm[k]), int(perm[(k + 1) % n]))) for k in range(n)}

    first = cycle_edges(rng.permutation(n))
    while True:
        second = cycle_edges(rng.permutation(n))
        if not (first & second):
            break
    adj: List[set] = [set() for _ in range(n)]
    for e in first | second:
        u, v = tuple(e)
        adj[u].add(v)
        adj[v].add(u)
    out = [sorted(s) for s in adj]
    assert all(len(s) == 4 for s in out)
    return out


# --------------------------------------------------------------------------------------
# Gossip matrices
# --------------------------------------------------------------------------------------
def metropolis_weights(adj: Adjacency) -> CSR:
    """Metropolis(-Hastings) weights: W_ij = 1/(1+max(deg_i, deg_j)) on edges, rest on the diagonal."""
    n = len(adj)
    deg = [len(a) for a in adj]
    m = np.zeros((n, n), dtype=np.float64)
    keep = np.zeros((n, n), dtype=bool)
    for i in range(n):
        for j in adj[i]:
            m[i, j] = 1.0 / (1.0 + max(deg[i], deg[j]))
            keep[i, j] = True
    for i in range(n):
        m[i, i] = 1.0 - m[i].sum()
        keep[i, i] = True
    return csr_from_dense(m, keep)


def average_consensus_matrix(n: int) -> CSR:
    """W* = 11^T / n (the paper's Average Consensus matrix)."""
    return csr_from_dense(np.full((n, n), 1.0 / n))


def slack_matrix(w0: CSR, kappa: float) -> CSR:
    """W_kappa = kappa*W0 + (1-kappa)*I (paper, Experiments section)."""
    m = kappa * w0.to_dense() + (1.0 - kappa) * np.eye(w0.n)
    keep = (w0.to_dense() != 0) | np.eye(w0.n, dtype=bool)
    return csr_from_dense(m, keep)


def directed_cycle_blend(n: int, self_w: float = 0.5, fwd_w: float = 0.3) -> CSR:
    """A NON-symmetric doubly stochastic matrix: self, i->i+1 and i->i-1 with unequal weights."""
    m = np.zeros((n, n))
    for i in range(n):
        m[i, i] += self_w
        m[i, (i + 1) % n] += fwd_w
        m[i, (i - 1) % n] += 1.0 - self_w - fwd_w
    return csr_from_dense(m)


# --------------------------------------------------------------------------------------
# Configurations
# --------------------------------------------------------------------------------------
@dataclass(frozen=True)
class Config:
    name: str
    n: int
    d: int
    K: int  # accelerated-gossip rounds per step (the paper's phase length R)
    alpha: float
    steps: int
    sigma: float
    seed: int
    graph: str  # "ring" | "torus8x8" | "regular4"
    a_dist: Tuple[str, float, float]  # ("uniform"|"loguniform", lo, hi)
    c_std: float
    mu_rule: str  # "linear" | "normal:<std>" | "sin4" | "uniform:<lo>:<hi>"
    x0_std: float  # 0 => x0 = 0; otherwise one N(0, std^2) draw per coordinate shared by all workers

    def with_d(self, d: int) -> "Config":
        return Config(**{**self.__dict__, "d": int(d)})

    def with_steps(self, steps: int) -> "Config":
        return Config(**{**self.__dict__, "steps": int(steps)})

    @property
    def wc(self) -> int:
        """Worker-coordinates touched by one step."""
        return self.n * self.d


CONFIGS: Dict[str, Config] = {
    "cfg1": Config("cfg1", 8, 4096, 2, 0.05, 10, 0.1, 0, "ring", ("uniform", 0.5, 2.0), 1.0, "linear", 0.0),
    "cfg2": Config("cfg2", 16, 270_000, 4, 0.01, 100, 0.1, 1, "ring", ("uniform", 0.5, 2.0), 1.0, "normal:2", 0.01),
    "cfg3": Config("cfg3", 64, 11_200_000, 8, 0.005, 50, 0.05, 2, "torus8x8", ("uniform", 0.1, 10.0), 1.0,
                   "normal:1", 0.0),
    "cfg4": Config("cfg4", 256, 1_000_000, 16, 0.002, 50, 0.1, 3, "ring", ("uniform", 0.5, 2.0), 0.5, "sin4", 0.0),
    "cfg5": Config("cfg5", 32, 25_600_000, 6, 0.001, 20, 0.1, 4, "regular4", ("loguniform", 0.01, 100.0), 1.0,
                   "uniform:-5:5", 0.0),
}


def gossip_matrix(cfg: Config) -> CSR:
    """The config's gossip matrix W (symmetric for all five configs)."""
    if cfg.graph == "ring":
        return metropolis_weights(ring_graph(cfg.n))
    if cfg.graph == "torus8x8":
        assert cfg.n == 64
        return metropolis_weights(torus_graph(8, 8))
    if cfg.graph == "regular4":
        return metropolis_weights(random_regular4_graph(cfg.n, cfg.seed))
    raise ValueError(cfg.graph)


def _block_rng(seed: int, stream: int, worker: int, block: int) -> np.random.Generator:
    key1 = (np.uint64(stream) << np.uint64(48)) | (np.uint64(worker) << np.uint64(28)) | np.uint64(block)
    return np.random.Generator(np.random.Philox(key=[np.uint64(seed), key1]))


def worker_means(cfg: Config) -> np.ndarray:
    """mu_i, the centre of worker i's targets c_ij (float64, length n)."""
    i = np.arange(cfg.n, dtype=np.float64)
    rule = cfg.mu_rule.split(":")
    if rule[0] == "linear":
        return i - (cfg.n - 1) / 2.0
    if rule[0] == "sin4":
        return 4.0 * np.sin(2.0 * math.pi * i / cfg.n)
    rng = _block_rng(cfg.seed, _STREAM_MU, 0, 0)
    if rule[0] == "normal":
        return float(rule[1]) * rng.standard_normal(cfg.n)
    if rule[0] == "uniform":
        lo, hi = float(rule[1]), float(rule[2])
        return lo + (hi - lo) * rng.random(cfg.n)
    raise ValueError(cfg.mu_rule)


def _draw_a(cfg: Config, worker: int, block: int, count: int) -> np.ndarray:
    kind, lo, hi = cfg.a_dist
    u = _block_rng(cfg.seed, _STREAM_A, worker, block).random(count)
    if kind == "uniform":
        return lo + (hi - lo) * u
    if kind == "loguniform":
        return np.exp(math.log(lo) + (math.log(hi) - math.log(lo)) * u)
    raise ValueError(kind)


def _fill_block(cfg: Config, mu: np.ndarray, block: int, lo: int, hi: int, j0: int,
                a: np.ndarray, c: np.ndarray, x0: np.ndarray) -> None:
    """Fill coordinates [lo, hi) of `block` into the output views (whose column 0 is coordinate j0)."""
    b0 = block * BLOCK
    cnt = min(BLOCK, cfg.d - b0)
    s0, s1 = lo - b0, hi - b0
    o0, o1 = lo - j0, hi - j0
    for i in range(cfg.n):
        a[i, o0:o1] = _draw_a(cfg, i, block, cnt)[s0:s1]
        z = _block_rng(cfg.seed, _STREAM_C, i, block).standard_normal(cnt)
        c[i, o0:o1] = (mu[i] + cfg.c_std * z)[s0:s1]
    if cfg.x0_std > 0.0:
        z = _block_rng(cfg.seed, _STREAM_X0, 0, block).standard_normal(cnt)
        x0[:, o0:o1] = (cfg.x0_std * z)[s0:s1].astype(np.float32)[None, :]
    else:
        x0[:, o0:o1] = 0.0


def objective_data(cfg: Config, j0: int = 0, j1: Optional[int] = None, threads: int = 1,
                   out: Optional[Tuple[np.ndarray, np.ndarray, np.ndarray]] = None
                   ) -> Tuple[np.ndarray, np.ndarray, np.ndarray]:
    """(a, c, x0) as float32 arrays of shape [n, j1-j0] for coordinates j0 <= j < j1.

    ``out`` may hold three preallocated float32 arrays (e.g. views of pinned host memory) with
    at least j1-j0 columns; only those columns are written.
    """
    j1 = cfg.d if j1 is None else j1
    if not (0 <= j0 <= j1 <= cfg.d):
        raise ValueError("coordinate range outside [0, d]")
    w = j1 - j0
    if out is None:
        a = np.empty((cfg.n, w), dtype=np.float32)
        c = np.empty((cfg.n, w), dtype=np.float32)
        x0 = np.empty((cfg.n, w), dtype=np.float32)
    else:
        a, c, x0 = out
    mu = worker_means(cfg)
    jobs = []
    if w > 0:
        for block in range(j0 // BLOCK, (j1 - 1) // BLOCK + 1):
            lo = max(j0, block * BLOCK)
            hi = min(j1, (block + 1) * BLOCK)
            jobs.append((block, lo, hi))
    if threads <= 1 or len(jobs) <= 1:
        for block, lo, hi in jobs:
            _fill_block(cfg, mu, block, lo, hi, j0, a, c, x0)
    else:
        with ThreadPoolExecutor(max_workers=threads) as ex:
            list(ex.map(lambda job: _fill_block(cfg, mu, job[0], job[1], job[2], j0, a, c, x0), jobs))
    return a, c, x0
