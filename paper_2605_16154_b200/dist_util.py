"""Helpers for running one process per GPU.

Default: independent replicas.  Every rank works on its own batch, no data-path collective; torch.distributed only
synchronises the start / end of the timed region and takes the slowest rank's time.

Data parallel (the paper's own runs used two GPUs, App. E): the ranks share ONE rollout batch.  Selection runs
replicated (it is a few kilobytes), the kept chunks are dealt out by trajectory, round-robin, every rank runs pack
and the actor update on its share under the global loss scale, and one all-reduce (sum) over the flat fp32
gradient buffer gives every rank the full-batch gradient.  Index bookkeeping only: no step of the method runs here.
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


def owned_trajectories(n_traj: int, rank: int, world_size: int) -> torch.Tensor:
    """Boolean mask [n_traj]: trajectory i belongs to rank i % world_size."""
    return (torch.arange(n_traj) % int(world_size)) == int(rank)


def partition_kept(kept_idx: torch.Tensor, kept_off: torch.Tensor, rank: int, world_size: int):
    """This rank's share of a selection.  kept_idx [>= n_kept] and kept_off [n_traj + 1] are the outputs of
    pcm_sample_chunks (any device).  Returns (idx_local [n_local] int32, off_local [n_traj + 1] int32): the kept
    chunk ids of the owned trajectories in their original order, and offsets in which every other trajectory has
    an empty segment, so that trajectory i of the batch is still trajectory i for the pack step."""
    dev = kept_off.device
    n_traj = kept_off.numel() - 1
    off = kept_off.to(torch.int64)
    m = off[1:] - off[:-1]
    mine = owned_trajectories(n_traj, rank, world_size).to(dev)
    m_local = torch.where(mine, m, torch.zeros_like(m))
    off_local = torch.zeros(n_traj + 1, dtype=torch.int64, device=dev)
    off_local[1:] = torch.cumsum(m_local, 0)
    n_kept = int(off[-1].item())
    slots = torch.arange(n_kept, device=dev)
    owner = torch.searchsorted(off[1:].contiguous(), slots, right=True)          # trajectory of every kept slot
    idx_local = kept_idx[:n_kept][mine[owner]].to(torch.int32).contiguous()
    return idx_local, off_local.to(torch.int32).contiguous()


def local_kept_count(lengths, budget: int, rank: int, world_size: int) -> int:
    """Kept chunks this rank will own: sum of min(budget, N_i) over its trajectories (known before sampling)."""
    total = 0
    for i, n in enumerate(lengths):
        if i % int(world_size) == int(rank):
            total += min(int(budget), int(n))
    return total


def allreduce_sum(flat: torch.Tensor) -> torch.Tensor:
    """Sum over all ranks, in place, of one flat tensor (the gradient buffer); identity without a process group."""
    if dist.is_available() and dist.is_initialized() and dist.get_world_size() > 1:
        dist.all_reduce(flat, op=dist.ReduceOp.SUM)
    return flat
