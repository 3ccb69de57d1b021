"""Host-side plumbing for running the path on several GPUs.

The folded quantized linear layer has no cross-token and no cross-batch dependency (Sec. 3.3: the
activation step is per token, the weight pack is a constant), so the path does not shard: every GPU
holds the whole folded weight pack and runs its own batches.  Nothing crosses NVLink on the data
path; the only collective is the MAX of the ranks' device-timed durations that the benchmark
reports.  This module holds that bookkeeping so that it can be exercised on CPU ranks (gloo).
"""
from __future__ import annotations

import os
from dataclasses import dataclass


@dataclass(frozen=True)
class RankInfo:
    rank: int
    world: int
    local_rank: int

    @staticmethod
    def from_env(env=None) -> "RankInfo":
        env = os.environ if env is None else env
        return RankInfo(int(env.get("RANK", "0")), int(env.get("WORLD_SIZE", "1")), int(env.get("LOCAL_RANK", "0")))


def replica_seed(base_seed: int, rank: int) -> int:
    """Each replica draws its own batches: distinct seeds per rank, the same for a given rank."""
    return base_seed + 7919 * rank


def split_batches(n_batches: int, world: int, rank: int) -> range:
    """Contiguous share of ``n_batches`` independent batches for ``rank`` (sizes differ by at most one)."""
    if world < 1 or not 0 <= rank < world or n_batches < 0:
        raise ValueError("bad rank layout")
    lo = (n_batches * rank) // world
    hi = (n_batches * (rank + 1)) // world
    return range(lo, hi)


def max_over_ranks(value: float, dist=None, device=None) -> float:
    """MAX of a per-rank scalar (a duration) over the process group; identity without a group."""
    if dist is None:
        return float(value)
    import torch
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def sum_over_ranks(value: float, dist=None, device=None) -> float:
    if dist is None:
        return float(value)
    import torch
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.SUM)
    return float(t.item())


def job_throughput(units_this_rank: float, seconds_this_rank: float, dist=None, device=None) -> float:
    """Whole-job rate: the units all ranks processed divided by the slowest rank's duration."""
    total = sum_over_ranks(units_this_rank, dist, device)
    slowest = max_over_ranks(seconds_this_rank, dist, device)
    return total / slowest
