"""Gaussian-kernel similarity (Section 4 item 2) on the GPU against the oracle.

The kernel values are fp32 on the GPU and double in the oracle; for int8 features the squared
distances are exact integers on both sides, so the only differences are the fp32 bandwidth factor
and expf (relative 1e-6); for bf16 features the fp32 dot products add about 1e-6 absolute to the
exponent.  Partitions are compared with the same teacher-forced rule as the cosine configurations.
"""
import numpy as np
import pytest

pytestmark = pytest.mark.gpu

OBJ_RTOL = 1e-4
PICK_RTOL = 1e-3


@pytest.fixture(scope="module")
def rcd():
    from paper_2211_00839_b200 import binding
    return binding


@pytest.fixture(scope="module")
def orc():
    from oracle import rcd_oracle
    return rcd_oracle


@pytest.mark.parametrize("name,M,d,batch", [("C1", 200, 64, 2), ("C2", 333, 512, 1), ("C4", 257, 256, 2), ("C3", 130, 37, 1)])
def test_gaussian_similarity_matches_oracle(rcd, orc, name, M, d, batch):
    import torch
    from paper_2211_00839_b200.workloads import make_workload
    wl = make_workload(name, L=batch, M=M, d=d, shuffle=False)
    with rcd.Context(0) as ctx:
        X = rcd.features_to_torch(wl.features, device=torch.device("cuda", 0)).view(batch, M, d)
        S, sigma = ctx.rcd_similarity_gaussian(X)
        ctx.sync_status()
        S, sigma = S.cpu().numpy(), sigma.cpu().numpy()
    for b in range(batch):
        want, sg = orc.similarity_gaussian(wl.features[b * M:(b + 1) * M])
        assert sigma[b] == pytest.approx(sg, rel=2e-6)
        assert np.allclose(S[b, :, :M], want, rtol=2e-5, atol=1e-7)
        assert np.all(np.diag(S[b, :, :M]) == 1.0)
        assert np.array_equal(S[b, :, :M], S[b, :, :M].T)
        assert np.all(S[b, :, M:] == 0)


def test_gaussian_similarity_of_coincident_points(rcd):
    import torch
    X = torch.full((1, 40, 128), 3, dtype=torch.int8, device="cuda")
    with rcd.Context(0) as ctx:
        S, sigma = ctx.rcd_similarity_gaussian(X)
        ctx.sync_status()
        assert float(sigma[0]) == 0.0 and bool((S[0, :, :40] == 1).all())


@pytest.mark.parametrize("name,L,M,d,path", [("C1", 2, 200, 64, 0), ("C2", 2, 700, 128, 0), ("C4", 3, 400, 256, 1)])
def test_partition_with_gaussian_similarity(rcd, orc, name, L, M, d, path):
    import torch
    from paper_2211_00839_b200.workloads import make_workload
    wl = make_workload(name, L=L, M=M, d=d)
    dev = torch.device("cuda", 0)
    with rcd.Context(0, similarity_kind=rcd.RCD_SIM_GAUSSIAN, greedy_path=path) as ctx:
        X = rcd.features_to_torch(wl.features, device=dev)
        y = torch.from_numpy(wl.labels).to(dev)
        a, o, v = ctx.rcd_partition(X, y, wl.capacities, wl.L)
        vals, total = ctx.rcd_objective(X, y, a, wl.W, wl.L)
        ctx.sync_status()
        assert v.dtype == torch.float64 and vals.dtype == torch.float64
        a, o, v, vals = a.cpu().numpy(), o.cpu().numpy(), v.cpu().numpy(), vals.cpu().numpy()
    assert np.allclose(v, vals, rtol=OBJ_RTOL)
    groups = orc.split_by_label(wl.labels, wl.L)
    off = 0
    for l, ids in enumerate(groups):
        Ml = len(ids)
        q = orc.quotas(Ml, wl.capacities)
        assert np.array_equal(np.bincount(a[ids], minlength=wl.W), q)
        picked = o[off:off + Ml]
        off += Ml
        local = np.searchsorted(ids, picked).astype(np.int32)
        S, _ = orc.similarity_gaussian(wl.features[ids])
        bad, stats, fv = orc.replay_class(S, q, a[picked], local, PICK_RTOL)
        assert bad == -1, (l, bad, stats)
        assert np.allclose(v[l], fv, rtol=OBJ_RTOL, atol=1e-9)
    want = orc.objective(wl.features, wl.labels, a, wl.W, wl.L, similarity_kind="gaussian")
    assert np.allclose(vals, want, rtol=1e-5, atol=1e-7)
