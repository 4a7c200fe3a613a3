"""Multi-GPU use of the compaction path: units (layer, sequence, KV head) are independent, so ranks take disjoint
sets of sequences and never exchange data. The only cross-rank step is the reduction of a timing or a counter."""
from __future__ import annotations

import numpy as np


def partition_sequences(lengths, world_size: int):
    """Longest-first greedy split of a batch's sequences into `world_size` shards of similar token count.
    Returns a list (one entry per rank) of ascending sequence indices; every sequence appears exactly once."""
    lengths = np.asarray(lengths, np.int64)
    order = np.argsort(-lengths, kind="stable")
    load = np.zeros(world_size, np.int64)
    shards = [[] for _ in range(world_size)]
    for s in order:
        r = int(np.argmin(load))
        shards[r].append(int(s))
        load[r] += int(lengths[s])
    return [sorted(s) for s in shards]


def shard_range(n_items: int, rank: int, world_size: int):
    """Contiguous balanced split of range(n_items): the half-open range of `rank`."""
    lo = n_items * rank // world_size
    hi = n_items * (rank + 1) // world_size
    return lo, hi


def max_over_ranks(value: float, device=None) -> float:
    """MAX-reduce a scalar over the default process group (a no-op without one)."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()):
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def sum_over_ranks(value: float, device=None) -> float:
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()):
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.SUM)
    return float(t.item())


def head_shard(Hq: int, Hkv: int, rank: int, world_size: int):
    """Head-sharded (tensor-parallel) layer: the half-open ranges of KV heads and of query heads that `rank` holds.
    KV heads are split contiguously and a KV head's query heads stay with it."""
    if Hkv % world_size or Hq % Hkv:
        raise ValueError("the KV heads must divide evenly over the ranks and the query heads over the KV heads")
    per, G = Hkv // world_size, Hq // Hkv
    return (rank * per, (rank + 1) * per), (rank * per * G, (rank + 1) * per * G)


def allreduce_headsum(u_heads):
    """The exchange between ta_score_headsum and ta_compress_from_headsum: an fp32 SUM all-reduce of the per-shard
    head sums [L][total_tokens] over the default process group, in place (a no-op without one)."""
    import torch.distributed as dist
    if dist.is_available() and dist.is_initialized():
        dist.all_reduce(u_heads, op=dist.ReduceOp.SUM)
    return u_heads
