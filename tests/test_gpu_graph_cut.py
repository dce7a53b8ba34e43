"""Algorithm 1 with the graph-cut objective (Section 4 item 2) on the GPU against the oracle.

int8 features with dot-product similarity: bit-exact.  bf16 / Gaussian similarity: the teacher-forced
rule of the facility-location tests (picks inside a 1e-3 relative gap, values within 1e-4)."""
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


def run(rcd, wl, **cfg):
    import torch
    dev = torch.device("cuda", 0)
    with rcd.Context(0, objective=rcd.RCD_OBJ_GRAPH_CUT, **cfg) as ctx:
        X = rcd.features_to_torch(wl.features, device=dev)
        y = torch.from_numpy(wl.labels).to(dev)
        a, o, v = ctx.rcd_partition(X, y, wl.capacities, wl.L)
        vals, total = ctx.rcd_objective(X, y, a, wl.W, wl.L)
        ctx.sync_status()
        return a.cpu().numpy(), o.cpu().numpy(), v.cpu().numpy(), vals.cpu().numpy(), total.cpu().numpy()


@pytest.mark.parametrize("name,kw", [("C1", {}), ("C2", dict(L=3, M=900, d=128)), ("C5", dict(L=4, M=333, d=75))])
def test_graph_cut_int8_exact(rcd, orc, name, kw):
    from paper_2211_00839_b200.workloads import make_workload
    wl = make_workload(name, **kw)
    a, o, v, vals, total = run(rcd, wl)
    ref = orc.partition(wl.features, wl.labels, wl.capacities, wl.L, variant="incremental", objective="cut")
    assert np.array_equal(a, ref.assignment)
    assert np.array_equal(o, ref.order)
    assert v.dtype == np.int64 and np.array_equal(v, ref.part_values)
    assert np.array_equal(vals, v) and total[0] == v.sum()       # tracked f == f from the definition
    if name == "C1":
        plain = orc.partition(wl.features, wl.labels, wl.capacities, wl.L, variant="plain", objective="cut")
        assert np.array_equal(a, plain.assignment) and np.array_equal(v, plain.part_values)


def test_graph_cut_ragged_classes(rcd, orc):
    from paper_2211_00839_b200.workloads import Workload
    rng = np.random.default_rng(8)
    sizes = [70, 0, 3, 400, 1]
    feats = rng.integers(-9, 10, size=(sum(sizes), 24)).astype(np.int8)
    labels = np.concatenate([np.full(m, l, np.int32) for l, m in enumerate(sizes)])
    perm = rng.permutation(len(labels))
    wl = Workload("ragged", "int8", np.ascontiguousarray(feats[perm]), np.ascontiguousarray(labels[perm]),
                  np.array([1.0, 2.0, 1.5, 1.0, 3.0]), len(sizes), 5)
    a, o, v, vals, total = run(rcd, wl)
    ref = orc.partition(wl.features, wl.labels, wl.capacities, wl.L, variant="plain", objective="cut")
    assert np.array_equal(a, ref.assignment) and np.array_equal(o, ref.order) and np.array_equal(v, ref.part_values)
    assert np.array_equal(vals, v)


@pytest.mark.parametrize("name,kw,sim", [("C4", dict(L=3, M=300, d=128), "dot"), ("C1", dict(L=2, M=150, d=32), "gaussian")])
def test_graph_cut_float_teacher_forced(rcd, orc, name, kw, sim):
    from paper_2211_00839_b200.workloads import make_workload
    wl = make_workload(name, **kw)
    a, o, v, vals, total = run(rcd, wl, similarity_kind=rcd.RCD_SIM_GAUSSIAN if sim == "gaussian" else rcd.RCD_SIM_DOT)
    assert v.dtype == np.float64
    assert np.allclose(vals, v, rtol=OBJ_RTOL, atol=1e-6)
    groups = orc.split_by_label(wl.labels, wl.L)
    off = 0
    for l, ids in enumerate(groups):
        M = len(ids)
        q = orc.quotas(M, wl.capacities)
        assert np.array_equal(np.bincount(a[ids], minlength=wl.W), q)
        picked = o[off:off + M]
        off += M
        local = np.searchsorted(ids, picked).astype(np.int32)
        S = orc.class_similarity(wl.features[ids], sim)
        bad, stats, fv = orc.replay_class(S, q, a[picked], local, PICK_RTOL, objective="cut")
        assert bad == -1, (l, bad, stats)
        assert np.allclose(v[l], fv, rtol=OBJ_RTOL, atol=1e-6)
    want = orc.objective(wl.features, wl.labels, a, wl.W, wl.L, similarity_kind=sim, objective="cut")
    assert np.allclose(vals, want, rtol=1e-5, atol=1e-6)
