"""Replica bookkeeping for runs on several GPUs of one node.

The attention JVP has no exchange step between GPUs: every (batch, head, query row) is independent, so a
multi-GPU run is N independent replicas of the single-GPU call.  The only cross-rank logic is how a timed
region is accounted: bracket it with a barrier on both sides, take the maximum device time over the ranks,
and divide the work of ALL ranks by it.  That logic lives here so that it can be exercised with the gloo
backend on CPUs.
"""
from __future__ import annotations

import torch


def max_over_ranks(value: float, dist=None, device=None) -> float:
    """Maximum of a per-rank scalar over all ranks (identity without a process group)."""
    if dist is None or not dist.is_initialized() or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def aggregate_throughput(work_per_rank: float, ms_this_rank: float, steps: int, dist=None, device=None):
    """Whole-job throughput of N replicas: (N * work per step) / (slowest rank's time per step).

    Returns (work_per_second, ms_per_step, world_size).
    """
    world = 1 if dist is None or not dist.is_initialized() else dist.get_world_size()
    total_ms = max_over_ranks(ms_this_rank, dist, device)
    ms_per_step = total_ms / steps
    return world * work_per_rank / (ms_per_step * 1e-3), ms_per_step, world
