"""Request sharding across ranks.

The refresh path has no cross-request data dependence: scores, the anchor set, the recomputed
rows, the private K/V and the attention of one request need only the weights and the shared
affix cache (Section 3.2, 4.1 of the paper).  So N ranks split the requests, replicate weights
and affix cache, and exchange nothing on the per-step path; ``torch.distributed`` is used
only for the timing barrier and the max over ranks.
"""
from __future__ import annotations

import socket
import sys
from typing import List, Sequence, Tuple


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


def free_port() -> int:
    """A TCP port on 127.0.0.1 that is free right now (for the rendezvous of a self-started run)."""
    with socket.socket() as sk:
        sk.bind(("127.0.0.1", 0))
        return int(sk.getsockname()[1])


def torchrun_command(script: str, argv: Sequence[str], n_ranks: int, port: int) -> List[str]:
    """The command that starts ``script argv`` as ``n_ranks`` ranks of one node, one per GPU, with the rendezvous on
    127.0.0.1 (the container's host name may not resolve)."""
    if n_ranks < 1:
        raise ValueError(n_ranks)
    return [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={n_ranks}",
            "--master-addr", "127.0.0.1", "--master-port", str(port), script, *argv]


def launch_plan(gpus: int, env) -> Tuple[str, int]:
    """What a process started as ``--gpus N`` has to do, from its environment:
    ("run", world)   it is a rank of a started job (WORLD_SIZE set and equal to N), or N == 1: run;
    ("spawn", N)     N > 1 and no job around it: start N ranks of itself;
    ("refuse", w)    WORLD_SIZE is set but differs from N: the line would describe a job that is not running."""
    world = env.get("WORLD_SIZE")
    if world is None:
        return ("run", 1) if gpus <= 1 else ("spawn", gpus)
    world = int(world)
    return ("run", world) if world == gpus else ("refuse", world)
