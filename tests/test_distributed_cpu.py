"""The class-sharded multi-rank path on CPU: two gloo ranks, the oracle standing in for the GPU
library as each rank's single-device partitioner."""
import os
import socket

import numpy as np
import pytest


def test_shard_classes_balances_cubic_work():
    from paper_2211_00839_b200.distributed import shard_classes
    shards = shard_classes([100, 100, 100, 100], 2)
    assert sorted(sum(shards, [])) == [0, 1, 2, 3] and [len(s) for s in shards] == [2, 2]
    shards = shard_classes([10, 500, 20, 30, 400], 2)
    assert sorted(sum(shards, [])) == [0, 1, 2, 3, 4]
    assert shards[0] == [1] and shards[1] == [0, 2, 3, 4]       # the 500^3 class alone outweighs the rest
    assert shard_classes([5, 0, 7], 4) == [[2], [0], [1], []]
    assert shard_classes([], 3) == [[], [], []]


def _worker(rank, world, port, out_dir):
    import torch.distributed as dist
    from oracle import rcd_oracle as orc
    from paper_2211_00839_b200.distributed import partition_sharded
    from paper_2211_00839_b200.workloads import make_workload
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        wl = make_workload("C1", L=5, M=40, d=16, seed=3)

        def single_device(features, labels, caps, L):
            return orc.partition(features, labels, caps, L, variant="incremental").assignment

        got = partition_sharded(wl.features, wl.labels, wl.capacities, wl.L, single_device)
        np.save(os.path.join(out_dir, "rank%d.npy" % rank), got)

        # the tensor form (the one the GPU path uses, here on CPU tensors over gloo)
        import torch
        from paper_2211_00839_b200.distributed import partition_sharded_tensors

        def single_device_t(f, y, caps, L):
            return torch.from_numpy(orc.partition(f.numpy(), y.numpy(), caps, L, variant="incremental").assignment)

        got_t = partition_sharded_tensors(torch.from_numpy(wl.features), torch.from_numpy(wl.labels), wl.capacities, wl.L,
                                          single_device_t)
        np.save(os.path.join(out_dir, "rank%d_t.npy" % rank), got_t.numpy())
    finally:
        dist.destroy_process_group()


def test_two_ranks_reproduce_the_single_process_partition(tmp_path):
    import torch.multiprocessing as mp
    from oracle import rcd_oracle as orc
    from paper_2211_00839_b200.workloads import make_workload
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    mp.spawn(_worker, args=(2, port, str(tmp_path)), nprocs=2, join=True)
    wl = make_workload("C1", L=5, M=40, d=16, seed=3)
    want = orc.partition(wl.features, wl.labels, wl.capacities, wl.L, variant="incremental").assignment
    for r in range(2):
        got = np.load(os.path.join(str(tmp_path), "rank%d.npy" % r))
        assert np.array_equal(got, want)
        got_t = np.load(os.path.join(str(tmp_path), "rank%d_t.npy" % r))
        assert np.array_equal(got_t, want)
