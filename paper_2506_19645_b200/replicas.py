"""Host-side plumbing for running one independent replica of the workload per GPU.

The path has no exchange step between GPUs (the tensor-parallel ranks are simulated inside
each GPU), so N GPUs run N replicas: no data-path collective.  What is shared is only the
clock: every rank times the same number of steps between two barriers and the job's time is
the maximum over ranks.
"""
from __future__ import annotations

import os

import torch
import torch.distributed as dist


def rank_env() -> tuple[int, int, int]:
    """(rank, local_rank, world_size) as torch.distributed.run exports them; (0, 0, 1) when run alone."""
    return (int(os.environ.get("RANK", "0")), int(os.environ.get("LOCAL_RANK", "0")),
            int(os.environ.get("WORLD_SIZE", "1")))


def barrier() -> None:
    if dist.is_available() and dist.is_initialized():
        dist.barrier()


def max_over_ranks(ms: float, device="cpu") -> float:
    """The slowest rank's time (identity when not running distributed)."""
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(ms)
    t = torch.tensor([float(ms)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_rate(units_per_replica_step: int, steps: int, world: int, ms_max: float) -> float:
    """Units (tokens) all replicas processed per second: world * units * steps / slowest rank's time."""
    return world * units_per_replica_step * steps / (ms_max * 1e-3)
