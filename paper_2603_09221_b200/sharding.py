"""Multi-GPU plumbing of the benchmark: instances are independent, so ranks never exchange data.

Every rank solves its own copy of the workload (weak scaling, a different seed per rank); the only
communication is one MAX-reduction of the elapsed time after the timed region.  This module holds that
logic so that it can be exercised on CPU ranks (gloo) as well as on GPUs (nccl).
"""
from __future__ import annotations

import os
import socket
import subprocess
import sys

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


def launcher_command(nproc: int, script: str, script_args, port: int | None = None):
    """Command line that starts `nproc` ranks of `script` on this node, one process per GPU: torch's elastic launcher
    with a rendezvous on 127.0.0.1 (the container hostname may not resolve) on a free port."""
    if port is None:
        with socket.socket() as sk:
            sk.bind(("127.0.0.1", 0))
            port = sk.getsockname()[1]
    return [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", str(int(nproc)),
            "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(script)] + list(script_args)


def launch_ranks(nproc: int, script: str, script_args, env=None) -> int:
    """Run `launcher_command` to completion; returns the launcher's exit code.  NCCL prints its version line so that
    the communicator (and with it the rank count) shows in the log."""
    env = dict(os.environ if env is None else env)
    env.setdefault("NCCL_DEBUG", "VERSION")
    return subprocess.call(launcher_command(nproc, script, script_args), env=env)
