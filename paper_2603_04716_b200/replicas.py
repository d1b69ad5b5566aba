"""Replica bookkeeping for multi-GPU runs.

The measured path does not shard: the allocation model treats instances as independent
replicas (Eq. 2-3 are linear in the instance counts), so N GPUs run N independent copies of
the measurement and only the timings are combined.  This module holds that combination: the
slowest rank's time (max over ranks) and the whole-job throughput over all replicas.  It uses
torch.distributed only for the all-reduce of a handful of doubles (NCCL on GPUs, gloo on CPU).
"""
from __future__ import annotations


def max_over_ranks(values, dist=None, device=None):
    """Element-wise maximum of a list of floats over all ranks (identity without a process group)."""
    if dist is None or not dist.is_initialized() or dist.get_world_size() == 1:
        return [float(v) for v in values]
    import torch
    t = torch.tensor([float(v) for v in values], dtype=torch.float64, device=device or "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return t.tolist()


def replica_throughput(units_per_rank: float, seconds_per_rank: float, dist=None, device=None):
    """Whole-job throughput of `world` replicas that each process `units_per_rank` units:
    world * units / (max over ranks of the time).  Returns (throughput, max_seconds, world)."""
    world = dist.get_world_size() if dist is not None and dist.is_initialized() else 1
    (t_max,) = max_over_ranks([seconds_per_rank], dist, device)
    return world * units_per_rank / t_max, t_max, world
