"""The multi-rank plumbing (replicas only: barrier + max-over-ranks timing, head sharding) on CPU
with two gloo ranks."""
import os
import socket

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
        out.put((rank, agg, seed, heads))
        dist.barrier()
    finally:
        dist.destroy_process_group()


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
    for rank, agg, seed, heads in results:
        assert agg == [15.0, 3.0]                            # max over ranks, element-wise
        assert seed == 4 + 1000 * rank
    assert results[0][3] == list(range(0, 14)) and results[1][3] == list(range(14, 28))
    assert replicas.whole_job_rate(7.15e12, 6.0, 2) == pytest.approx(2 * 7.15e12 / 6e-3)


def test_single_process_is_identity_and_bad_shard_is_rejected():
    assert replicas.max_over_ranks([1.5, 2.5]) == [1.5, 2.5]
    assert list(replicas.shard_heads(32, 32, 4, 3)) == list(range(24, 32))
    with pytest.raises(ValueError):
        replicas.shard_heads(28, 4, 3, 0)
