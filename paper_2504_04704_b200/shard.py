"""Multi-GPU sharding of the compress pass: host logic only.

Every (sequence, layer, KV head) is independent (Section 2.2 scores and selects per head and
per partition), so ranks take disjoint caches and the data path has no collective.  The only
communication is the bookkeeping of a measurement: the slowest rank's time.
"""
from __future__ import annotations

import torch
import torch.distributed as dist


def rank_seed(base_seed: int, rank: int) -> int:
    """Seed of one layer's cache on one rank: ranks hold different synthetic caches."""
    return int(base_seed) + 100000 * int(rank)


def shard_units(total_units: int, rank: int, world: int) -> range:
    """Contiguous share of ``total_units`` independent (b, h) units for ``rank`` (strong-scaling
    split of one cache; sizes differ by at most one)."""
    lo = total_units * rank // world
    hi = total_units * (rank + 1) // world
    return range(lo, hi)


def max_over_ranks(value: float, device=None) -> float:
    """Largest ``value`` over all ranks (the job is as slow as its slowest rank)."""
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def job_throughput(units_per_rank: int, world: int, ms_slowest: float) -> float:
    """Whole-job units per second when every rank processes ``units_per_rank`` (weak scaling)."""
    return world * units_per_rank / (ms_slowest * 1e-3)
