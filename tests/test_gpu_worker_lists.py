"""Per-worker index lists and batch sizes (Algorithm 2's initialisation) against the oracle, through the C ABI."""
import numpy as np
import pytest

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def rcd():
    import torch
    if not torch.cuda.is_available():
        pytest.skip("needs a CUDA device")
    from paper_2211_00839_b200 import binding
    return binding


@pytest.fixture(scope="module")
def orc():
    from oracle import rcd_oracle
    return rcd_oracle


@pytest.mark.parametrize("N,W,seed", [(1, 1, 0), (7, 3, 1), (1023, 4, 2), (1024, 64, 3), (5000, 9, 4), (70001, 1024, 5)])
def test_worker_lists_match_the_definition(rcd, orc, N, W, seed):
    """Bit-exact: several chunks of the stable split, a ragged tail, workers that get nothing."""
    import torch
    rng = np.random.default_rng(seed)
    a = rng.integers(0, max(1, W - 1), size=N).astype(np.int32)      # the last worker stays empty when W > 1
    with rcd.Context(0) as ctx:
        off, idx = rcd.rcd_worker_lists(ctx, torch.from_numpy(a).cuda(), W)
        ctx.sync_status()
        off, idx = off.cpu().numpy(), idx.cpu().numpy()
    want_off, want_idx = orc.worker_lists(a, W)
    assert np.array_equal(off, want_off)
    assert np.array_equal(idx, want_idx)


def test_worker_lists_of_a_partition(rcd, orc):
    """From rcd_partition's own output: list sizes are the quota sums over the classes."""
    import torch
    from paper_2211_00839_b200.workloads import make_workload
    wl = make_workload("C2", L=3, M=700)
    with rcd.Context(0) as ctx:
        X = rcd.features_to_torch(wl.features, device=torch.device("cuda", 0))
        y = torch.from_numpy(wl.labels).cuda()
        a, _, _ = ctx.rcd_partition(X, y, wl.capacities, wl.L)
        off, idx = rcd.rcd_worker_lists(ctx, a, wl.W)
        ctx.sync_status()
        a, off, idx = a.cpu().numpy(), off.cpu().numpy(), idx.cpu().numpy()
    want_off, want_idx = orc.worker_lists(a, wl.W)
    assert np.array_equal(off, want_off) and np.array_equal(idx, want_idx)
    q = orc.quotas(700, wl.capacities)
    assert (off[1:] - off[:-1]).tolist() == (3 * q).tolist()


def test_worker_lists_reject_a_bad_block_number(rcd):
    import torch
    a = torch.tensor([0, 1, 5, 1], dtype=torch.int32).cuda()
    with rcd.Context(0) as ctx:
        with pytest.raises(rcd.RcdError) as e:
            rcd.rcd_worker_lists(ctx, a, 3)
        assert e.value.status == 1
        off, idx = rcd.rcd_worker_lists(ctx, a, 6)          # the context stays usable
        assert off.cpu().tolist() == [0, 1, 3, 3, 3, 3, 4]


def test_batch_sizes_match_the_oracle(rcd, orc):
    for B, r in ((32, [1, 1, 2, 4]), (10, [4, 1, 3]), (1, [8, 1]), (64, [1.0, 2.5, 3.5]), (128, [3.0, 0.7, 1.9, 5.2])):
        assert rcd.rcd_batch_sizes(B, r).tolist() == orc.batch_sizes(B, r).tolist()
    with pytest.raises(rcd.RcdError):
        rcd.rcd_batch_sizes(0, [1, 2])
    with pytest.raises(rcd.RcdError):
        rcd.rcd_batch_sizes(8, [1, -2])
