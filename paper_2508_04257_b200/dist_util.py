"""Multi-GPU plumbing of the benchmark: the path shards by sequence with no data-path exchange, so ranks only need a
rendezvous, a barrier, and a max-over-ranks of their device times (torch.distributed; NCCL on GPUs, gloo on CPU)."""
from __future__ import annotations

import os
from dataclasses import dataclass

import torch
import torch.distributed as dist


@dataclass
class RankInfo:
    rank: int
    world: int
    local_rank: int


def rank_info() -> RankInfo:
    return RankInfo(int(os.environ.get("RANK", "0")), int(os.environ.get("WORLD_SIZE", "1")), int(os.environ.get("LOCAL_RANK", "0")))


def rank_seed(base_seed: int, rank: int) -> int:
    """Every rank draws its own batch of sequences (weak scaling: per-rank work is fixed)."""
    return base_seed + 7919 * rank


def max_over_ranks(value: float, device) -> float:
    """The slowest rank's time; a single-process run returns the value unchanged."""
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def aggregate_throughput(units_per_rank: float, world: int, seconds_max: float) -> float:
    """Whole-job throughput: the units all ranks processed divided by the slowest rank's time."""
    return world * units_per_rank / seconds_max
