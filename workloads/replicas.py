"""Replica bookkeeping for runs on several GPUs (plain torch.distributed, no arithmetic of the method).

The attention path has no exchange step: sequences are independent, so N GPUs run N independent
replicas of the workload on different seeded inputs.  The only communication is the barrier around
the timed region and the maximum over ranks of the measured time; the job's throughput is the
work of all replicas divided by the slowest replica's time.
"""
from __future__ import annotations

import os


def dist_env():
    """(rank, local_rank, world_size) from the launcher's environment (single process if absent)."""
    return int(os.environ.get("RANK", 0)), int(os.environ.get("LOCAL_RANK", 0)), int(os.environ.get("WORLD_SIZE", 1))


def replica_seed(base_seed: int, rank: int) -> int:
    """Each replica draws its own inputs."""
    return int(base_seed) + 17 * int(rank)


def max_over_ranks(value: float, world: int, device="cpu") -> float:
    """Maximum of a per-rank scalar (the job is as slow as its slowest replica)."""
    if world <= 1:
        return float(value)
    import torch
    import torch.distributed as dist
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def job_throughput(units_per_replica_step: float, ms_per_step: float, world: int) -> float:
    """Whole-job units per second: every replica does the same work per step (weak scaling)."""
    return world * units_per_replica_step / (ms_per_step * 1e-3)
