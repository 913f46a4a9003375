"""Rank bookkeeping of a multi-GPU run.

The layer does not shard: N GPUs run N independent replicas of the same work (one process per GPU, no
collective on the data path).  What the ranks do share is the clock of a measurement: a timed region is
bracketed by barriers, every rank measures its own duration on its device, and the job's duration is the
maximum over the ranks.  These helpers are the whole of it; they work on any torch.distributed backend
(NCCL on GPUs, gloo on CPUs in the tests).
"""
from __future__ import annotations


def max_over_ranks(seconds: float, device=None) -> float:
    """Duration of the job: the slowest rank's.  No-op without an initialised process group."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(seconds)
    t = torch.tensor([seconds], dtype=torch.float64, device=device if device is not None else "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def job_throughput(units_per_rank: float, world: int, job_seconds: float) -> float:
    """Units the whole job processed per second: every replica does `units_per_rank` in `job_seconds`."""
    return world * units_per_rank / job_seconds


def barrier():
    import torch.distributed as dist
    if dist.is_available() and dist.is_initialized() and dist.get_world_size() > 1:
        dist.barrier()
