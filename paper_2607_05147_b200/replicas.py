"""Host-side logic of multi-GPU runs.  The path does not shard across GPUs: requests are
independent and the scheduler is per engine, so N GPUs run N independent replicas (one process
per GPU) with no data-path collective.  What the ranks do share is bookkeeping: distinct seeds,
a barrier around the timed region, the max over ranks of the device time, the whole-job rate."""
from __future__ import annotations

import os
from typing import Sequence

import torch


def env_ranks():
    """(rank, local_rank, world_size) from the torchrun environment (1 process: 0, 0, 1)."""
    return (int(os.environ.get("RANK", "0")), int(os.environ.get("LOCAL_RANK", "0")),
            int(os.environ.get("WORLD_SIZE", "1")))


def rank_seed(base: int, rank: int, k: int) -> int:
    """Seed of the k-th synthetic batch of a rank: replicas never verify the same tensors."""
    return base + 97 * rank + k


def max_over_ranks(values: Sequence[float], dist=None, device="cpu"):
    """Element-wise max over all ranks of a few floats (device times in ms)."""
    if dist is None:
        return [float(v) for v in values]
    t = torch.tensor(list(values), dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(x) for x in t]


def whole_job_rate(units_per_rank_per_step: int, steps: int, ms: float, world: int) -> float:
    """Units per second over all replicas: every rank does the same amount of work per step (weak
    scaling), the job takes as long as its slowest rank."""
    return world * units_per_rank_per_step * steps / (ms * 1e-3)


def is_reporting_rank(rank: int) -> bool:
    return rank == 0
