"""Multi-GPU plumbing of the benchmark: instances are independent, so ranks never exchange data.

Every rank solves its own copy of the workload (weak scaling, a different seed per rank); the only
communication is one MAX-reduction of the elapsed time after the timed region.  This module holds that
logic so that it can be exercised on CPU ranks (gloo) as well as on GPUs (nccl).
"""
from __future__ import annotations

import torch
import torch.distributed as dist

from . import workloads


def rank_seed(cfg_id: int, rank: int) -> int:
    """Seed of the workload generator on `rank` (rank 0 uses the configuration's own seed)."""
    return workloads.SEED0 + cfg_id + 1000 * rank


def max_over_ranks(value: float, device="cpu") -> float:
    """MAX of a per-rank scalar over all ranks (identity without a process group)."""
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([value], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def aggregate_throughput(instances_per_rank: int, ms_per_step_local: float, device="cpu"):
    """Whole-job throughput: all ranks' instances divided by the slowest rank's time.

    Returns (instances_per_second, ms_per_step_max, world_size)."""
    world = dist.get_world_size() if (dist.is_available() and dist.is_initialized()) else 1
    ms = max_over_ranks(ms_per_step_local, device)
    return world * instances_per_rank / (ms * 1e-3), ms, world
