"""The class-sharded path with the CUDA library as the per-rank partitioner (one rank: no collective; the two-rank
exchange is covered on CPU over gloo by tests/test_distributed_cpu.py with the same code)."""
import numpy as np
import pytest

pytestmark = pytest.mark.gpu


def test_sharded_partition_on_one_gpu_equals_the_direct_call_and_the_oracle():
    import torch
    from oracle import rcd_oracle as orc
    from paper_2211_00839_b200 import binding as rcd
    from paper_2211_00839_b200.distributed import partition_sharded_gpu
    from paper_2211_00839_b200.workloads import make_workload
    dev = torch.device("cuda", 0)
    wl = make_workload("C2", L=5, M=400, d=128)
    X = rcd.features_to_torch(wl.features, device=dev)
    y = torch.from_numpy(wl.labels).to(dev)
    with rcd.Context(0) as ctx:
        direct, _, _ = ctx.rcd_partition(X, y, wl.capacities, wl.L)
        sharded = partition_sharded_gpu(ctx, X, y, wl.capacities, wl.L)
        ctx.sync_status()
        assert sharded.is_cuda and torch.equal(direct, sharded)
    want = orc.partition(wl.features, wl.labels, wl.capacities, wl.L, variant="incremental").assignment
    assert np.array_equal(sharded.cpu().numpy(), want)


def test_sharded_partition_of_a_subset_of_classes_on_the_gpu():
    """What a rank of a two-rank job does with its shard (the classes shard_classes gives rank 1), on the GPU:
    equal to the oracle's partition of those classes."""
    import torch
    from oracle import rcd_oracle as orc
    from paper_2211_00839_b200 import binding as rcd
    from paper_2211_00839_b200.distributed import shard_classes
    from paper_2211_00839_b200.workloads import make_workload
    dev = torch.device("cuda", 0)
    wl = make_workload("C2", L=5, M=300, d=64)
    mine = shard_classes(np.bincount(wl.labels, minlength=wl.L).tolist(), 2)[1]
    keep = np.isin(wl.labels, mine)
    remap = -np.ones(wl.L, dtype=np.int32)
    remap[mine] = np.arange(len(mine), dtype=np.int32)
    feats, labs = np.ascontiguousarray(wl.features[keep]), remap[wl.labels[keep]]
    with rcd.Context(0) as ctx:
        a, _, _ = ctx.rcd_partition(rcd.features_to_torch(feats, device=dev), torch.from_numpy(labs).to(dev), wl.capacities, len(mine))
        ctx.sync_status()
    want = orc.partition(wl.features, wl.labels, wl.capacities, wl.L, variant="incremental").assignment[keep]
    assert np.array_equal(a.cpu().numpy(), want)
