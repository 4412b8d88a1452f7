"""Host-side helpers for running the path on several GPUs.

The path has no exchange step between ranks: every rank quantizes its own workers' buckets, so a
multi-GPU run is a set of independent replicas that only meet for timing (weak scaling).  These two
helpers are all the cross-rank logic there is; they work with any torch.distributed backend, which
lets the CPU tests cover them with gloo.
"""
from __future__ import annotations

from typing import List


def worker_ids(rank: int, workers_per_rank: int) -> List[int]:
    """Global ids (= data seeds) of the simulated workers that `rank` owns; disjoint across ranks."""
    return [rank * workers_per_rank + k for k in range(workers_per_rank)]


def max_over_ranks(value: float, dist=None, device=None) -> float:
    """The slowest rank's value (a step time): what a multi-GPU throughput has to be computed from."""
    if dist is None or not dist.is_initialized() or dist.get_world_size() == 1:
        return float(value)
    import torch

    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def aggregate_throughput(bytes_per_rank: float, ms_per_step_max: float, world_size: int) -> float:
    """Whole-job GB/s: every rank moved `bytes_per_rank` in the time of the slowest rank."""
    return world_size * bytes_per_rank / (ms_per_step_max * 1e-3) / 1e9
