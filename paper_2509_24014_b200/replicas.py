"""Helpers for running the path on several GPUs of one node.

The path has no exchange step: every (batch, query head) is independent and patterns are per
head, so N GPUs either run N independent replicas, or split one layer's heads between them
(whole grouped-query groups, so no K/V head is duplicated). Neither needs a collective on the
data path; the only cross-rank traffic is for timing (a barrier around the timed region and a
max over ranks of the measured times). Works with any torch.distributed backend (nccl on GPUs,
gloo on CPU).

Head sharding: a rank calls the ordinary library entry points on views of Q, K, V, O restricted
to its heads (head-offset pointers with the tensors' own strides: no copies) and keeps a pattern
of its own, whose row_ptr counts from zero. `merge_shard_patterns` puts such per-rank CSR arrays
back into the single-device row order ((b * heads_q + h) * num_blocks + query block) on the host.
"""
from __future__ import annotations

import dataclasses
from typing import List, Optional, Sequence, Tuple

import numpy as np
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


def shard_kv_heads(heads_kv: int, world: int, rank: int) -> range:
    """K/V heads owned by `rank` (the groups of shard_heads)."""
    if heads_kv % world != 0:
        raise ValueError("heads_kv must be divisible by the number of ranks")
    per = heads_kv // world
    return range(rank * per, (rank + 1) * per)


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


def merge_shard_patterns(shards: Sequence[Tuple[Sequence[int], np.ndarray, np.ndarray]], batch: int, heads_q: int,
                         num_blocks: int) -> Tuple[np.ndarray, np.ndarray]:
    """Assembles per-rank CSR patterns into the single-device one.

    shards: one (heads, row_ptr, col_idx) per rank; `heads` are the rank's query heads in ascending
    order, row_ptr / col_idx its local CSR with rows ordered ((b * len(heads) + local head) *
    num_blocks + query block) and row_ptr[0] == 0. Returns (row_ptr, col_idx) with rows ordered
    ((b * heads_q + h) * num_blocks + query block). Every head must belong to exactly one shard."""
    owner = {}
    for si, (heads, _, _) in enumerate(shards):
        for j, h in enumerate(heads):
            if h in owner:
                raise ValueError(f"query head {h} is in two shards")
            owner[int(h)] = (si, j)
    if sorted(owner) != list(range(heads_q)):
        raise ValueError("the shards do not cover every query head exactly once")
    row_ptr = np.zeros(batch * heads_q * num_blocks + 1, dtype=np.int64)
    pieces = []
    r = 0
    for b in range(batch):
        for h in range(heads_q):
            si, j = owner[h]
            heads, rp, ci = shards[si]
            lo = (b * len(heads) + j) * num_blocks
            seg = np.asarray(rp[lo:lo + num_blocks + 1], dtype=np.int64)
            pieces.append(np.asarray(ci[seg[0]:seg[-1]]))
            row_ptr[r + 1:r + num_blocks + 1] = row_ptr[r] + (seg[1:] - seg[0])
            r += num_blocks
    col_idx = np.concatenate(pieces) if pieces else np.zeros(0, dtype=np.int32)
    return row_ptr.astype(np.int32), col_idx.astype(np.int32)


@dataclasses.dataclass
class HeadShard:
    """One rank's share of a layer whose heads are split over `world` ranks: which heads it owns,
    its own pattern buffers (row_ptr counts from zero) and its workspace."""
    world: int
    rank: int
    heads: range
    kv_heads: range
    params: object
    pattern: object
    row_ptr: torch.Tensor
    col_idx: torch.Tensor
    ws: torch.Tensor

    def views(self, q, k, v, o):
        """Views of the full-layer tensors [B, H, L, D] restricted to this rank's heads (no copies)."""
        hq, hkv = self.heads, self.kv_heads
        return (q[:, hq.start:hq.stop], k[:, hkv.start:hkv.stop], v[:, hkv.start:hkv.stop], o[:, hq.start:hq.stop])


def plan_head_shard(batch: int, heads_q: int, heads_kv: int, seq_len: int, params, world: int, rank: int,
                    device) -> HeadShard:
    """Allocates the pattern buffers and the switch-step workspace for rank `rank` of `world`."""
    from . import binding as sd
    heads = shard_heads(heads_q, heads_kv, world, rank)
    kv_heads = shard_kv_heads(heads_kv, world, rank)
    nb = seq_len // params.block_size
    k_pre, k_gen = sd.sparsed_kept_per_row(params, seq_len)
    pat, row_ptr, col_idx = sd.new_pattern(batch, len(heads), nb, k_pre + k_gen, device)
    shape = sd.Shape(batch, len(heads), len(kv_heads), seq_len, 128)
    ws = sd.new_workspace(sd.sparsed_workspace_bytes(sd.OP_ATTENTION_STEP, shape, params), device)
    return HeadShard(world, rank, heads, kv_heads, params, pat, row_ptr, col_idx, ws)


def head_shard_step(shard: HeadShard, q, k, v, o, step_1based: int, total_steps: int, skip: float,
                    softmax_scale: float = 0.0) -> int:
    """Algorithm 1's step for this rank's heads: sparsed_attention_step on head-offset views of the
    full-layer tensors q, o [B, Hq, L, D] and k, v [B, Hkv, L, D] (same strides, no copies, no
    collective). A rank that holds only its own heads calls sparsed_attention_step on them directly
    with shard.pattern and shard.ws. Returns the mode that ran."""
    from . import binding as sd
    qs, ks, vs, os_ = shard.views(q, k, v, o)
    return sd.sparsed_attention_step(qs, ks, vs, os_, shard.params, step_1based, total_steps, skip, shard.pattern,
                                     shard.ws, softmax_scale=softmax_scale)
