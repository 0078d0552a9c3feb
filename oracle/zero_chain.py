"""Float64 CPU oracle of the zero-chain objective and its Bernoulli-progress gradient oracle.

TEST INFRASTRUCTURE ONLY: used by tests.  Shares no code with the CUDA path and never imports it.

Source: "Optimal Complexity in Decentralized Training" (arXiv 2006.08085), proof of Theorem 1, the equation
defining the base zero-chain function fhat, and "Setting 1" there (every worker holds fhat itself; the oracle
multiplies the first not-yet-reached coordinate's partial derivative by z/p with z ~ Bernoulli(p); the final
rescaling f(x) = (L lambda^2 / l_1) fhat(x / lambda)).

Readings (the source text is garbled at two places):
  * Phi is printed with exp(+t^2/2) under the integral, which diverges; the function the proof relies on (its
    stated bounds Delta_0 = 12, l_1 = 152, G_inf = 23 hold for it) is
        Phi(z) = sqrt(e) * integral_{-inf}^{z} exp(-t^2/2) dt = sqrt(2 pi e) * N(z),   N = standard normal CDF.
  * The sum's second product is printed with a misplaced parenthesis; it is Psi(x_i) * Phi(x_{i+1}).
So, with x_0 := 1 (which turns the leading term into the i = 0 term of the sum, as Psi(-1) = 0):
        fhat(x) = sum_{i=0}^{T-1} [ Psi(-x_i) Phi(-x_{i+1}) - Psi(x_i) Phi(x_{i+1}) ]
        Psi(z) = exp(1 - 1/(2z-1)^2) for z > 1/2, else 0.
Coordinates are 1..T in the paper, 0..T-1 in the arrays here; prog(x) = number of leading coordinates up to and
including the last non-zero one (0 for x = 0).
"""
from __future__ import annotations

import math

import numpy as np

from .philox import philox4x32_10

SQRT_E = math.sqrt(math.e)


def psi(z: np.ndarray) -> np.ndarray:
    z = np.asarray(z, dtype=np.float64)
    out = np.zeros_like(z)
    m = z > 0.5
    out[m] = np.exp(1.0 - 1.0 / (2.0 * z[m] - 1.0) ** 2)
    return out


def psi_prime(z: np.ndarray) -> np.ndarray:
    z = np.asarray(z, dtype=np.float64)
    out = np.zeros_like(z)
    m = z > 0.5
    u = 2.0 * z[m] - 1.0
    out[m] = np.exp(1.0 - 1.0 / u ** 2) * 4.0 / u ** 3
    return out


def phi(z: np.ndarray) -> np.ndarray:
    z = np.asarray(z, dtype=np.float64)
    erfc = np.vectorize(math.erfc, otypes=[np.float64])
    return SQRT_E * math.sqrt(2.0 * math.pi) * 0.5 * erfc(-z / math.sqrt(2.0))


def phi_prime(z: np.ndarray) -> np.ndarray:
    z = np.asarray(z, dtype=np.float64)
    return SQRT_E * np.exp(-0.5 * z * z)


def value(x: np.ndarray) -> np.ndarray:
    """fhat of every row of x ([n, T])."""
    x = np.asarray(x, dtype=np.float64)
    prev = np.concatenate([np.ones((x.shape[0], 1)), x[:, :-1]], axis=1)  # x_{i} for the term that holds x_{i+1}
    return (psi(-prev) * phi(-x) - psi(prev) * phi(x)).sum(axis=1)


def gradient(x: np.ndarray) -> np.ndarray:
    """Exact gradient of fhat for every row of x: coordinate j collects the term in which it is the Phi argument
    (with its left neighbour in Psi) and the term in which it is the Psi argument (with its right neighbour in Phi)."""
    x = np.asarray(x, dtype=np.float64)
    prev = np.concatenate([np.ones((x.shape[0], 1)), x[:, :-1]], axis=1)
    g = -(psi(-prev) * phi_prime(-x) + psi(prev) * phi_prime(x))
    nxt = x[:, 1:]
    g[:, :-1] -= psi_prime(-x[:, :-1]) * phi(-nxt) + psi_prime(x[:, :-1]) * phi(nxt)
    return g


def prog(x: np.ndarray) -> np.ndarray:
    """Per row: index (1-based) of the last non-zero coordinate, 0 if there is none."""
    x = np.asarray(x)
    nz = x != 0
    idx = np.where(nz, np.arange(1, x.shape[1] + 1)[None, :], 0)
    return idx.max(axis=1)


def bernoulli_draws(seed: int, t: int, n: int, p: float) -> np.ndarray:
    """z_i in {0, 1} for workers 0..n-1 at step t: Philox4x32-10 with key (seed low, seed high) and counter
    (i, 0, 0xB0B0B0B0, t); z = 1 iff (first word + 0.5) * 2^-32 < p."""
    i = np.arange(n, dtype=np.uint64)
    r = philox4x32_10(i, np.uint64(0), np.uint64(0xB0B0B0B0), np.uint64(t), seed & 0xFFFFFFFF, (seed >> 32) & 0xFFFFFFFF)
    u = (r[0].astype(np.float64) + 0.5) * 2.0 ** -32
    return (u < p).astype(np.float64)


def stochastic_gradient(x: np.ndarray, lam: float, gain: float, p: float, seed: int, t: int) -> np.ndarray:
    """The rescaled oracle of Setting 1: g_i(x) = gain * ghat_i(x / lam) with
    [ghat_i(u)]_j = d_j fhat(u) * (1 + 1{j > prog(u)} (z_i / p - 1)),  z_i ~ Bernoulli(p);
    gain = L * lam / l_1 in the paper."""
    u = np.asarray(x, dtype=np.float64) / lam
    g = gradient(u)
    z = bernoulli_draws(seed, t, u.shape[0], p)
    beyond = np.arange(1, u.shape[1] + 1)[None, :] > prog(u)[:, None]
    factor = np.where(beyond, (z / p)[:, None], 1.0)
    return gain * g * factor
