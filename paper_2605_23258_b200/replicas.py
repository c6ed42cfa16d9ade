"""Replica bookkeeping for runs on several GPUs.

The hot path has no exchange step: units (sequence, layer, KV head) are independent in every call, so
N GPUs run N independent replicas of a workload and nothing crosses NVLink on the data path.  What is
shared is only the clock: a multi-GPU number is the work of all replicas over the slowest replica's
device time.  These helpers are the whole multi-rank logic; they run on any torch.distributed backend
(NCCL on GPUs, gloo in the CPU tests).
"""
from __future__ import annotations

import torch
import torch.distributed as dist


def world() -> tuple[int, int]:
    """(rank, world size); (0, 1) when no process group is up."""
    if dist.is_available() and dist.is_initialized():
        return dist.get_rank(), dist.get_world_size()
    return 0, 1


def slowest(times_ms, device="cpu") -> list[float]:
    """Element-wise maximum over ranks of a list of device times."""
    t = torch.tensor(list(times_ms), dtype=torch.float64, device=device)
    if world()[1] > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return t.tolist()


def aggregate_throughput(units_per_replica: float, time_ms: float, device="cpu") -> float:
    """Whole-job throughput: the units all replicas processed over the slowest replica's time."""
    (t,) = slowest([time_ms], device)
    return world()[1] * units_per_replica / (t * 1e-3)
