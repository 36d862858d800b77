"""Helpers for running independent replicas, one process per GPU.

The hot path does not shard: every rank works on its own batch and no data-path collective is needed.
torch.distributed only synchronises the start / end of the timed region and takes the slowest rank's time.
"""
from __future__ import annotations

import torch
import torch.distributed as dist


def replica_seed(base_seed: int, rank: int) -> int:
    """Seed of the batch rank `rank` works on (distinct batches, same distribution)."""
    return int(base_seed) + 1000 * int(rank)


def max_over_ranks(value: float, device) -> float:
    """Largest `value` over all ranks (the job is as slow as its slowest replica)."""
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def aggregate_throughput(units_per_rank: int, steps: int, elapsed_ms_max: float, world_size: int) -> float:
    """Whole-job units per second: every rank processed units_per_rank * steps units in elapsed_ms_max."""
    return world_size * units_per_rank * steps / (elapsed_ms_max / 1e3)
