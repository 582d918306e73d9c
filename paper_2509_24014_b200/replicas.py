"""Helpers for running the path on several GPUs of one node.

The path has no exchange step: every (batch, query head) is independent and patterns are per
head, so N GPUs run N independent replicas (or head shards chosen by the caller). The only
cross-rank traffic is for timing: a barrier around the timed region and a max over ranks of
the measured times. Works with any torch.distributed backend (nccl on GPUs, gloo on CPU).
"""
from __future__ import annotations

from typing import Dict, List, Optional, Sequence

import torch


def replica_seed(base_seed: int, rank: int) -> int:
    """Seed of the synthetic inputs of rank `rank` (replicas use different data)."""
    return int(base_seed) + 1000 * int(rank)


def shard_heads(heads_q: int, heads_kv: int, world: int, rank: int) -> range:
    """Query heads owned by `rank` when one layer is split over `world` ranks: whole GQA groups
    are kept together so that no K/V head is duplicated. Requires heads_kv % world == 0."""
    if heads_kv % world != 0:
        raise ValueError("heads_kv must be divisible by the number of ranks")
    group = heads_q // heads_kv
    per = heads_kv // world
    return range(rank * per * group, (rank + 1) * per * group)


def max_over_ranks(values: Sequence[float], dist=None, device="cpu") -> List[float]:
    """Element-wise maximum of `values` over all ranks (identity without a process group)."""
    if dist is None or not dist.is_initialized() or dist.get_world_size() == 1:
        return [float(v) for v in values]
    t = torch.tensor(list(values), dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return t.tolist()


def whole_job_rate(units_per_rank: float, ms: float, world: int) -> float:
    """Aggregate rate of `world` replicas that each processed `units_per_rank` in at most `ms`."""
    return world * units_per_rank / (ms * 1e-3)
