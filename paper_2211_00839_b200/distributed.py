"""Class-sharded partition over several ranks (one process per GPU).

Algorithm 1 treats every class on its own (it loops over V_1..V_L and joins the blocks at the
end), so the classes are the unit of sharding: each rank partitions its own classes with the
single-GPU library and one all-gather returns the full assignment.  There is no exchange while
the greedy loops run.
"""
from __future__ import annotations

from typing import Callable, List, Optional, Sequence

import numpy as np

__all__ = ["shard_classes", "partition_sharded", "partition_sharded_tensors", "partition_sharded_gpu"]


def shard_classes(class_sizes: Sequence[int], world: int) -> List[List[int]]:
    """Assign classes to ranks, balancing the greedy work (about M^3 per class): largest first,
    each to the least-loaded rank (ties to the lowest rank).  Deterministic."""
    load = [0] * world
    shards: List[List[int]] = [[] for _ in range(world)]
    order = sorted(range(len(class_sizes)), key=lambda l: (-int(class_sizes[l]), l))
    for l in order:
        r = min(range(world), key=lambda k: (load[k], k))
        shards[r].append(l)
        load[r] += int(class_sizes[l]) ** 3
    return [sorted(s) for s in shards]


def partition_sharded(features: np.ndarray, labels: np.ndarray, capacities: Sequence[float], L: int,
                      partition_fn: Callable[[np.ndarray, np.ndarray, Sequence[float], int], np.ndarray],
                      group=None, device: Optional[str] = None) -> np.ndarray:
    """Every rank calls this with the same inputs; returns the full assignment [N] on every rank.

    ``partition_fn(features, labels, capacities, L) -> assignment`` partitions a dataset on this
    rank (the GPU library in production).  ``device`` is where the gathered tensors live
    ("cuda:i" for NCCL, None/"cpu" for gloo)."""
    import torch
    import torch.distributed as dist

    rank = dist.get_rank(group)
    world = dist.get_world_size(group)
    labels = np.asarray(labels)
    sizes = np.bincount(labels, minlength=L)
    mine = shard_classes(sizes.tolist(), world)[rank]
    remap = -np.ones(L, dtype=np.int64)
    remap[mine] = np.arange(len(mine))
    idx = np.nonzero(remap[labels] >= 0)[0]                 # my samples, in dataset order
    if len(idx):
        local = partition_fn(np.ascontiguousarray(features[idx]), remap[labels[idx]].astype(np.int32),
                             capacities, max(len(mine), 1))
        local = np.asarray(local, dtype=np.int32)
    else:
        local = np.zeros(0, dtype=np.int32)

    # one all-gather of (index, block) pairs, padded to the largest shard
    dev = torch.device(device) if device else torch.device("cpu")
    n = torch.tensor([len(idx)], dtype=torch.int64, device=dev)
    counts = [torch.zeros_like(n) for _ in range(world)]
    dist.all_gather(counts, n, group=group)
    most = int(max(int(c.item()) for c in counts))
    pack = torch.full((2, max(most, 1)), -1, dtype=torch.int32, device=dev)
    if len(idx):
        pack[0, :len(idx)] = torch.from_numpy(idx.astype(np.int32)).to(dev)
        pack[1, :len(idx)] = torch.from_numpy(local).to(dev)
    packs = [torch.empty_like(pack) for _ in range(world)]
    dist.all_gather(packs, pack, group=group)
    out = np.full(len(labels), -1, dtype=np.int32)
    for c, p in zip(counts, packs):
        k = int(c.item())
        p = p.cpu().numpy()
        out[p[0, :k]] = p[1, :k]
    return out


def partition_sharded_tensors(features, labels, capacities: Sequence[float], L: int, partition_fn, group=None):
    """The same sharding with torch tensors that stay where they are (CUDA tensors with NCCL, CPU tensors with gloo).

    ``features`` [N, d] and ``labels`` [N] (int32) are the whole dataset, identical on every rank;
    ``partition_fn(features, labels, capacities, L) -> assignment`` (tensors on the same device) partitions this
    rank's classes.  Indices and blocks never leave the device: the class sizes are read back once (L integers,
    they fix the shards), this rank's samples are selected with a mask, and one all-gather of (index, block)
    pairs, padded to the largest shard, rebuilds the full assignment [N] on every rank.  With one rank there is
    no collective at all."""
    import torch
    import torch.distributed as dist

    world = dist.get_world_size(group) if dist.is_available() and dist.is_initialized() else 1
    rank = dist.get_rank(group) if world > 1 else 0
    dev = labels.device
    N = labels.numel()
    sizes = torch.bincount(labels.to(torch.int64), minlength=L).cpu().tolist()
    mine = shard_classes(sizes, world)[rank]
    remap = torch.full((max(L, 1),), -1, dtype=torch.int32)
    if mine:
        remap[torch.tensor(mine, dtype=torch.int64)] = torch.arange(len(mine), dtype=torch.int32)
    remap = remap.to(dev)
    local_label = remap[labels.to(torch.int64)]
    idx = torch.nonzero(local_label >= 0).flatten()                 # my samples, in dataset order
    if idx.numel():
        local = partition_fn(features.index_select(0, idx).contiguous(), local_label.index_select(0, idx).contiguous(),
                             capacities, max(len(mine), 1)).to(torch.int32)
    else:
        local = torch.zeros(0, dtype=torch.int32, device=dev)
    out = torch.full((N,), -1, dtype=torch.int32, device=dev)
    if world == 1:
        out[idx] = local
        return out
    counts = [int(sum(sizes[l] for l in shard)) for shard in shard_classes(sizes, world)]   # every rank knows every shard's size
    most = max(max(counts), 1)
    pack = torch.full((2, most), -1, dtype=torch.int32, device=dev)
    pack[0, :idx.numel()] = idx.to(torch.int32)
    pack[1, :idx.numel()] = local
    packs = [torch.empty_like(pack) for _ in range(world)]
    dist.all_gather(packs, pack, group=group)
    for k, p in zip(counts, packs):
        out[p[0, :k].to(torch.int64)] = p[1, :k]
    return out


def partition_sharded_gpu(ctx, features, labels, capacities: Sequence[float], L: int, group=None):
    """Class-sharded partition with the CUDA library as every rank's partitioner (``ctx``: this rank's
    ``binding.Context``; ``features`` / ``labels``: the whole dataset on this rank's GPU).  One NCCL all-gather of
    4-byte (index, block) pairs at the end; nothing is exchanged while the greedy loops run."""
    def on_this_gpu(f, y, caps, nclasses):
        assignment, _, _ = ctx.rcd_partition(f, y, caps, nclasses, want_order=False, want_values=False)
        return assignment
    return partition_sharded_tensors(features, labels, capacities, L, on_this_gpu, group=group)
