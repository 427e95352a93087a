"""Multi-GPU bookkeeping: replicas only.

The decode path of one request never leaves its GPU (the shared state, the record arena and the
ancestry index of a request live together, and requests are independent), so N GPUs run N independent
replicas of the workload with no data-path collective.  The only exchange is the timing protocol of the
benchmark: a barrier on both sides of the timed region and the maximum over ranks of each rank's
device-measured time.
"""
from __future__ import annotations

from typing import Sequence

import torch
import torch.distributed as dist


def world() -> tuple[int, int]:
    """(rank, world_size); (0, 1) when no process group is up."""
    if dist.is_available() and dist.is_initialized():
        return dist.get_rank(), dist.get_world_size()
    return 0, 1


def barrier() -> None:
    if dist.is_available() and dist.is_initialized():
        dist.barrier()


def max_over_ranks(values: Sequence[float], device="cpu") -> list[float]:
    """Element-wise maximum over ranks of a few scalars (each rank's own device-measured milliseconds)."""
    t = torch.tensor(list(values), dtype=torch.float64, device=device)
    if dist.is_available() and dist.is_initialized() and dist.get_world_size() > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(x) for x in t.cpu()]


def aggregate_throughput(units_per_rank_step: int, ms_per_step_max: float, world_size: int) -> float:
    """Whole-job units per second: every replica processed units_per_rank_step in the slowest rank's time."""
    return world_size * units_per_rank_step / (ms_per_step_max * 1e-3)
