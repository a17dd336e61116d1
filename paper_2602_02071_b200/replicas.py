"""Rank bookkeeping for multi-GPU runs.

The BAPS attention path has no exchange step: query tiles, heads and batches are independent, and
splitting the key axis would change results (the method is order dependent).  A multi-GPU run is
therefore N independent replicas; the only communication is a barrier and the maximum over ranks of
the device time, from which the whole-job throughput is computed.
"""
from __future__ import annotations

import os

import torch
import torch.distributed as dist


def dist_env():
    """(rank, world_size, local_rank) from the environment set by ``torch.distributed.run``."""
    return (int(os.environ.get("RANK", "0")), int(os.environ.get("WORLD_SIZE", "1")),
            int(os.environ.get("LOCAL_RANK", "0")))


def max_over_ranks(value: float, device: str = "cpu") -> float:
    """Largest ``value`` held by any rank (identity when no process group is initialised)."""
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_rate(work_per_rank: float, ms_per_step_max: float, world_size: int) -> float:
    """Aggregate rate of ``world_size`` replicas that each do ``work_per_rank`` per step, the step
    time being the slowest rank's."""
    return world_size * work_per_rank / (ms_per_step_max * 1e-3)
