"""Multi-GPU runs are independent replicas: every rank steps its own copy of the
workload (the path has no exchange between GPUs).  The only cross-rank work is
measurement: a barrier around the timed region, the maximum of the ranks'
device times, and the whole-job throughput computed from it."""
from __future__ import annotations

from typing import Optional

import torch
import torch.distributed as dist


def world_size() -> int:
    return dist.get_world_size() if dist.is_available() and dist.is_initialized() else 1


def barrier() -> None:
    if world_size() > 1:
        dist.barrier()


def max_over_ranks(value: float, device: Optional[torch.device] = None) -> float:
    """The largest `value` any rank reports (the slowest rank's time)."""
    if world_size() == 1:
        return float(value)
    t = torch.tensor([value], dtype=torch.float64, device=device or "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_throughput(local_ms: float, units_per_step: int, steps: int,
                         device: Optional[torch.device] = None) -> tuple:
    """(units/s summed over all replicas, max-over-ranks milliseconds).  Every rank
    processes units_per_step * steps units; the job takes as long as its slowest rank."""
    ms = max_over_ranks(local_ms, device)
    return world_size() * units_per_step * steps / (ms * 1e-3), ms
