"""Multi-GPU plumbing: the path does not shard, so N GPUs run N independent
replicas of the workload.  The only cross-rank steps are a barrier around the
timed region and the maximum of the per-rank times; both go through
``torch.distributed`` (NCCL on GPUs, gloo in the CPU tests)."""
from __future__ import annotations

import torch
import torch.distributed as dist


def world() -> int:
    return dist.get_world_size() if dist.is_available() and dist.is_initialized() else 1


def barrier() -> None:
    if world() > 1:
        dist.barrier()


def max_over_ranks(value: float, device: str | torch.device = "cpu") -> float:
    """Largest `value` over all ranks (the slowest replica sets the job's time)."""
    if world() == 1:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def job_throughput(units_per_rank: float, seconds_this_rank: float, device: str | torch.device = "cpu") -> float:
    """Whole-job throughput of independent replicas: every rank processed
    `units_per_rank`, the job took as long as its slowest rank."""
    return world() * units_per_rank / max_over_ranks(seconds_this_rank, device)
