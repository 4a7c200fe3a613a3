"""Host logic of the multi-GPU path on CPU: two gloo ranks split a ragged batch without overlap and reduce a
timing with MAX, as the benchmark does; and the head-sharded variant's bookkeeping: disjoint head ranges per rank and
an fp32 sum all-reduce of the per-shard head sums that leaves every rank with the same array."""
import os
import socket

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2604_11288_b200 import sharding


def test_partition_covers_and_balances():
    rng = np.random.default_rng(0)
    lengths = rng.integers(2048, 16385, size=64)
    for world in (1, 2, 4, 8):
        shards = sharding.partition_sequences(lengths, world)
        flat = sorted(i for s in shards for i in s)
        assert flat == list(range(64))
        loads = [int(lengths[s].sum()) for s in shards]
        assert max(loads) - min(loads) <= lengths.max()
    assert [sharding.shard_range(10, r, 4) for r in range(4)] == [(0, 2), (2, 5), (5, 7), (7, 10)]


def _worker(rank, world, port, lengths, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        mine = sharding.partition_sequences(lengths, world)[rank]
        gathered = [None] * world
        dist.all_gather_object(gathered, mine)
        t = sharding.max_over_ranks(1.0 + rank)
        tok = sharding.sum_over_ranks(float(sum(lengths[i] for i in mine)))
        if rank == 0:
            out.put((gathered, t, tok))
    finally:
        dist.destroy_process_group()


def test_two_ranks_gloo():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    lengths = [int(x) for x in np.random.default_rng(1).integers(100, 1000, size=9)]
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, lengths, q)) for r in range(2)]
    for p in procs:
        p.start()
    gathered, t, tok = q.get(timeout=120)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert sorted(gathered[0] + gathered[1]) == list(range(9))
    assert not set(gathered[0]) & set(gathered[1])
    assert t == 2.0 and tok == float(sum(lengths))


def test_head_shard_ranges():
    assert sharding.head_shard(32, 8, 0, 2) == ((0, 4), (0, 16))
    assert sharding.head_shard(32, 8, 1, 2) == ((4, 8), (16, 32))
    assert [sharding.head_shard(8, 4, r, 4)[0] for r in range(4)] == [(0, 1), (1, 2), (2, 3), (3, 4)]
    import pytest
    with pytest.raises(ValueError):
        sharding.head_shard(32, 8, 0, 3)


def _headsum_worker(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        (k0, k1), (q0, q1) = sharding.head_shard(8, 4, rank, world)
        # stand-in for ta_score_headsum: a per-head table summed over this rank's KV heads
        per_head = torch.arange(4 * 2 * 50, dtype=torch.float32).reshape(4, 2, 50) * 0.25  # [Hkv][L][total]
        mine = per_head[k0:k1].sum(dim=0)
        total = sharding.allreduce_headsum(mine.clone())
        out.put((rank, (k0, k1, q0, q1), total))
    finally:
        dist.destroy_process_group()


def test_headsum_allreduce_two_ranks_gloo():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    procs = [ctx.Process(target=_headsum_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    got = sorted([q.get(timeout=120) for _ in range(2)], key=lambda t: t[0])
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert got[0][1] == (0, 2, 0, 4) and got[1][1] == (2, 4, 4, 8)
    want = (torch.arange(4 * 2 * 50, dtype=torch.float32).reshape(4, 2, 50) * 0.25).sum(dim=0)
    assert torch.equal(got[0][2], want) and torch.equal(got[1][2], want)
