"""Rank plumbing for the benchmark: environment parsing and max-over-ranks timing.

The verify step does not shard (one GPU, no collective on the data path), so a
multi-GPU run is N independent replicas; the only exchange is this reduction of
the per-rank timings, done with torch.distributed (NCCL on GPUs, gloo on CPU).
"""
from __future__ import annotations

import os
from typing import Sequence

import torch
import torch.distributed as dist


def rank_info():
    """(rank, world_size, local_rank) from the torchrun environment (defaults 0, 1, 0)."""
    return (int(os.environ.get("RANK", "0")), int(os.environ.get("WORLD_SIZE", "1")),
            int(os.environ.get("LOCAL_RANK", "0")))


def max_over_ranks(values: Sequence[float], device: str = "cpu"):
    """Element-wise maximum of `values` over all ranks (identity when not distributed)."""
    t = torch.tensor(list(values), dtype=torch.float64, device=device)
    if dist.is_available() and dist.is_initialized() and dist.get_world_size() > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(x) for x in t.cpu()]


def aggregate_replicas(step_us_per_rank_max: float, world: int):
    """Whole-job throughput of `world` independent replicas that each finish a step in the
    (max over ranks) time: steps per second summed over all GPUs."""
    return world * 1e6 / step_us_per_rank_max
