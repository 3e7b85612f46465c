"""Host logic of the multi-GPU run: one independent cluster partition per rank.

The scheduling path shards by job with no exchange when every GPU schedules its own
partition of the cluster (its own jobs and its own cores).  What the ranks share is only
the timing protocol: a barrier on both sides of the timed region and the maximum over
ranks of the measured times.  `torch.distributed` does both (NCCL on GPUs, gloo in the
CPU tests).
"""

from __future__ import annotations

import os


def rank_info():
    """(rank, local_rank, world_size) from the launcher's environment (1 process if unset)."""
    return (int(os.environ.get("RANK", 0)), int(os.environ.get("LOCAL_RANK", 0)),
            int(os.environ.get("WORLD_SIZE", 1)))


def partition_seed_offset(rank: int) -> int:
    """Seed offset of a rank's partition: every rank draws different jobs, reproducibly."""
    return int(rank)


def max_over_ranks(values, device="cpu"):
    """Element-wise maximum of a list of floats over all ranks (identity without a process group)."""
    import torch
    import torch.distributed as dist
    t = torch.tensor(list(values), dtype=torch.float64, device=device)
    if dist.is_available() and dist.is_initialized() and dist.get_world_size() > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(v) for v in t.cpu()]


def whole_job_rate(units_per_rank: int, world_size: int, milliseconds: float) -> float:
    """Units all ranks processed per second, given the slowest rank's time per step."""
    return world_size * units_per_rank / (milliseconds * 1e-3)
