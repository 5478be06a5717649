"""Multi-GPU = independent replicas.

The decode-step path shards by sequence (each replica of a rollout pool owns its requests and their
KV cache) with no exchange inside attention or acceptance, so N GPUs run N copies of the step on
different batches.  The only cross-rank traffic is bookkeeping for the benchmark: a barrier around
the timed region and the maximum of the per-rank times.  These helpers hold that logic so that it
can be exercised on CPU with the gloo backend.
"""
from __future__ import annotations

from typing import Optional

import torch
import torch.distributed as dist


def rank_seed(base_seed: int, rank: int) -> int:
    """Every replica draws its own batch: the seed of rank r."""
    return int(base_seed) + int(rank)


def max_over_ranks(value: float, device: Optional[torch.device] = None) -> float:
    """Largest ``value`` across the process group (the job is as slow as its slowest replica)."""
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def sum_over_ranks(value: float, device: Optional[torch.device] = None) -> float:
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.SUM)
    return float(t.item())


def job_throughput(units_this_rank: float, ms_this_rank: float, device: Optional[torch.device] = None):
    """Whole-job throughput: units of all ranks divided by the slowest rank's time.

    Returns ``(units_per_second, total_units, max_ms)``.
    """
    total = sum_over_ranks(units_this_rank, device)
    ms = max_over_ranks(ms_this_rank, device)
    return total / (ms * 1e-3), total, ms
