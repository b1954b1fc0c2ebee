"""Multi-rank bookkeeping of the benchmark (one process per GPU, independent replicas).

The NVFP4 linear-layer path shards by tokens with no collective on the data path (the data-parallel all-reduce of
dW belongs to the trainer, not to this library), so N ranks are N replicas: the job's time is the slowest rank's,
its work the sum over ranks. Only the timing scalar crosses ranks."""
from __future__ import annotations

import torch
import torch.distributed as dist


def world_info():
    if dist.is_available() and dist.is_initialized():
        return dist.get_rank(), dist.get_world_size()
    return 0, 1


def max_over_ranks(value: float, device="cpu") -> float:
    """Largest `value` among all ranks (every rank gets it)."""
    _, world = world_info()
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    if world > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def job_throughput(units_per_rank: float, seconds_local: float, device="cpu") -> float:
    """Whole-job throughput: units of all ranks divided by the slowest rank's time."""
    _, world = world_info()
    return world * units_per_rank / max_over_ranks(seconds_local, device)
