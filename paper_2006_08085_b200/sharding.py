"""Multi-GPU decomposition of the DeTAG step: plumbing only.

The step never mixes coordinates (gossip mixes workers, the objective is diagonal), so ranks take
contiguous coordinate shards and the step needs no data-path collective.  Two scalars cross ranks:
the step time (MAX) and the consensus error (SUM of the per-shard sums of squares).
"""
from __future__ import annotations

from typing import Tuple


def shard_bounds(d_total: int, rank: int, world: int, align: int = 4) -> Tuple[int, int]:
    """Coordinates [j0, j1) of `rank`: contiguous, disjoint, covering [0, d_total); interior cuts on a
    multiple of `align` so every shard's row stays 16-byte aligned inside the global arrays."""
    if not (0 <= rank < world) or d_total < 0:
        raise ValueError("bad rank/world/d")
    per = -(-d_total // world)
    per = -(-per // align) * align
    j0 = min(rank * per, d_total)
    j1 = min(j0 + per, d_total)
    return j0, j1


def weak_scaling_offset(d_per_rank: int, rank: int) -> int:
    """Weak scaling: every rank steps a shard of d_per_rank coordinates; this is its global column 0
    (it enters the noise counter, so ranks draw different noise)."""
    return rank * d_per_rank


def reduce_max(value: float, dist, device=None) -> float:
    """MAX over ranks of a host scalar (step time): every rank reports the slowest rank's time."""
    import torch

    t = torch.tensor([value], dtype=torch.float64, device=device)
    if dist is not None and dist.is_initialized() and dist.get_world_size() > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def reduce_sum(value: float, dist, device=None) -> float:
    """SUM over ranks (per-shard consensus errors add up to the global one)."""
    import torch

    t = torch.tensor([value], dtype=torch.float64, device=device)
    if dist is not None and dist.is_initialized() and dist.get_world_size() > 1:
        dist.all_reduce(t, op=dist.ReduceOp.SUM)
    return float(t.item())
