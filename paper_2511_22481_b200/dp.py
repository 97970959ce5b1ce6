"""Data-parallel bookkeeping for decode replicas (one process per GPU).

Requests are independent, so ranks never exchange data on the decode path: each rank runs its own
batch against its own KV pool.  The only collectives are the ones a benchmark needs to report a
whole-job number: a barrier, the slowest rank's time, and the total units of work.
"""
from __future__ import annotations

from typing import Sequence

import torch
import torch.distributed as dist


def world() -> tuple[int, int]:
    """(rank, world_size); (0, 1) when no process group is initialised."""
    if dist.is_available() and dist.is_initialized():
        return dist.get_rank(), dist.get_world_size()
    return 0, 1


def shard_requests(num_requests: int, world_size: int, rank: int) -> range:
    """Contiguous, near-equal share of request ids for `rank` (strong-scaling helper: a request
    and its KV pages live on exactly one rank)."""
    if not 0 <= rank < world_size:
        raise ValueError("rank outside the world")
    base, extra = divmod(num_requests, world_size)
    start = rank * base + min(rank, extra)
    return range(start, start + base + (1 if rank < extra else 0))


def job_throughput(local_ms: Sequence[float], local_units: float, device=None) -> tuple[list[float], float]:
    """Reduce per-rank timings to whole-job numbers.

    local_ms     elapsed milliseconds of this rank's timed regions (any number of them)
    local_units  units of work (bytes, tokens) this rank processed per timed region
    Returns (max over ranks of each time, sum over ranks of the units).
    """
    t = torch.tensor(list(local_ms), dtype=torch.float64, device=device)
    u = torch.tensor([float(local_units)], dtype=torch.float64, device=device)
    _, n = world()
    if n > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        dist.all_reduce(u, op=dist.ReduceOp.SUM)
    return [float(x) for x in t.tolist()], float(u.item())
