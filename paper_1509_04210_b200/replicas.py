"""Rank plumbing for replica runs: one independent parameter server per GPU, no data-path collective.

The only cross-rank step is timing: a barrier on both sides of the timed region and the maximum
of the per-rank device times, from which the whole-job rate is formed.
"""
from __future__ import annotations

import os


def rank_info():
    """(rank, local_rank, world_size) from the launcher's environment; (0, 0, 1) when run alone."""
    return (int(os.environ.get("RANK", "0")), int(os.environ.get("LOCAL_RANK", "0")),
            int(os.environ.get("WORLD_SIZE", "1")))


def max_over_ranks(values, device="cpu"):
    """Element-wise maximum of a list of floats over all ranks (identity without a process group)."""
    import torch
    import torch.distributed as dist

    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return [float(v) for v in values]
    t = torch.tensor([float(v) for v in values], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(x) for x in t.cpu()]


def whole_job_rate(steps_per_rank, world_size, slowest_ms):
    """Units all ranks processed divided by the slowest rank's time (weak scaling)."""
    return world_size * steps_per_rank / (slowest_ms * 1e-3)


def replica_seed(master_seed, rank):
    """Every replica draws its own synthetic streams."""
    return int(master_seed) + int(rank)
