"""Request sharding across ranks.

The refresh path has no cross-request data dependence: scores, the anchor set, the recomputed
rows, the private K/V and the attention of one request need only the weights and the shared
affix cache (Section 3.2, 4.1 of the paper).  So N ranks split the requests, replicate weights
and affix cache, and exchange nothing on the per-step path; ``torch.distributed`` is used
only for the timing barrier and the max over ranks.
"""
from __future__ import annotations

from typing import Tuple


def shard_range(n_requests: int, rank: int, world: int) -> Tuple[int, int]:
    """Contiguous block [lo, hi) of requests owned by ``rank``; sizes differ by at most one."""
    if world <= 0 or not (0 <= rank < world) or n_requests < 0:
        raise ValueError((n_requests, rank, world))
    base, rem = divmod(n_requests, world)
    lo = rank * base + min(rank, rem)
    return lo, lo + base + (1 if rank < rem else 0)


def max_over_ranks(value: float, dist=None, device=None) -> float:
    """Max of a per-rank scalar (the step time) over all ranks; identity without a process group."""
    if dist is None or not dist.is_initialized() or dist.get_world_size() == 1:
        return float(value)
    import torch
    t = torch.tensor([float(value)], dtype=torch.float64, device=device or "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def aggregate_throughput(units_per_rank_step: int, world: int, ms_per_step_max: float) -> float:
    """Whole-job units per second: every rank's units over the slowest rank's step time."""
    return world * units_per_rank_step / (ms_per_step_max * 1e-3)
