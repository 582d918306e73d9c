"""The multi-rank plumbing (replicas only: barrier + max-over-ranks timing, head sharding) on CPU
with two gloo ranks."""
import os
import socket

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2509_24014_b200 import replicas


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        dist.barrier()
        local_ms = [10.0 + 5.0 * rank, 3.0 - rank]          # rank 0: (10, 3); rank 1: (15, 2)
        agg = replicas.max_over_ranks(local_ms, dist)
        seed = replicas.replica_seed(4, rank)
        heads = list(replicas.shard_heads(28, 4, world, rank))
        # head-sharded patterns: every rank builds the CSR of its own heads (row_ptr from zero), the ranks
        # exchange them as host objects, and the merged pattern must be the single-device one
        rp_g, ci_g, nb, batch = _global_pattern()
        mine = _local_pattern(rp_g, ci_g, heads, 28, nb, batch)
        gathered = [None] * world
        dist.all_gather_object(gathered, mine)
        rp_m, ci_m = replicas.merge_shard_patterns(gathered, batch, 28, nb)
        merged_ok = bool(np.array_equal(rp_m, rp_g) and np.array_equal(ci_m, ci_g))
        kv = list(replicas.shard_kv_heads(4, world, rank))
        out.put((rank, agg, seed, heads, merged_ok, kv))
        dist.barrier()
    finally:
        dist.destroy_process_group()


def _global_pattern():
    """A ragged single-device CSR over (batch 2, 28 heads, 6 query blocks) with seeded lists."""
    rng = np.random.default_rng(7)
    nb, batch = 6, 2
    lists = [sorted(rng.choice(nb, size=int(rng.integers(1, nb + 1)), replace=False).tolist())
             for _ in range(batch * 28 * nb)]
    rp = np.cumsum([0] + [len(x) for x in lists]).astype(np.int32)
    return rp, np.concatenate(lists).astype(np.int32), nb, batch


def _local_pattern(rp_g, ci_g, heads, heads_q, nb, batch):
    """What a rank that owns `heads` would hold: its rows only, row_ptr counting from zero."""
    lens, cols = [], []
    for b in range(batch):
        for h in heads:
            for ib in range(nb):
                r = (b * heads_q + h) * nb + ib
                lens.append(rp_g[r + 1] - rp_g[r])
                cols.append(ci_g[rp_g[r]:rp_g[r + 1]])
    return list(heads), np.cumsum([0] + lens).astype(np.int32), np.concatenate(cols).astype(np.int32)


def test_two_rank_replicas_over_gloo():
    world = 2
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, world, port, out)) for r in range(world)]
    for p in procs:
        p.start()
    results = sorted(out.get(timeout=120) for _ in range(world))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, agg, seed, heads, merged_ok, kv in results:
        assert agg == [15.0, 3.0]                            # max over ranks, element-wise
        assert seed == 4 + 1000 * rank
        assert merged_ok                                     # shard patterns line up with the global row order
        assert [h // 7 for h in heads] == sorted(kv * 7)     # whole GQA groups: each head's kv head is local
    assert results[0][3] == list(range(0, 14)) and results[1][3] == list(range(14, 28))
    assert sorted(results[0][3] + results[1][3]) == list(range(28))
    assert replicas.whole_job_rate(7.15e12, 6.0, 2) == pytest.approx(2 * 7.15e12 / 6e-3)


def test_single_process_is_identity_and_bad_shard_is_rejected():
    assert replicas.max_over_ranks([1.5, 2.5]) == [1.5, 2.5]
    assert list(replicas.shard_heads(32, 32, 4, 3)) == list(range(24, 32))
    with pytest.raises(ValueError):
        replicas.shard_heads(28, 4, 3, 0)
    rp_g, ci_g, nb, batch = _global_pattern()
    whole = _local_pattern(rp_g, ci_g, range(28), 28, nb, batch)
    rp_m, ci_m = replicas.merge_shard_patterns([whole], batch, 28, nb)
    assert np.array_equal(rp_m, rp_g) and np.array_equal(ci_m, ci_g)
    with pytest.raises(ValueError):                          # a head in two shards
        replicas.merge_shard_patterns([whole, _local_pattern(rp_g, ci_g, range(3), 28, nb, batch)], batch, 28, nb)
    with pytest.raises(ValueError):                          # a head in no shard
        replicas.merge_shard_patterns([_local_pattern(rp_g, ci_g, range(27), 28, nb, batch)], batch, 28, nb)
