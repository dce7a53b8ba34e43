"""Full-size configurations in the launch configuration bench.py times (default context).

The oracle cannot run these end to end in seconds, so outputs are sampled: whole classes where a
class is small enough (classes are independent in Algorithm 1, so a class of the big run must
equal the oracle's run of that class alone), a replayed prefix and single late picks where it is
not; plus properties that hold at any size (exact quotas, disjoint cover, tracked f equal to f
recomputed from the final assignment).
"""
import importlib.util
import json
import os
from concurrent.futures import ThreadPoolExecutor

import numpy as np
import pytest

pytestmark = pytest.mark.gpu

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _golden_module():
    """The script that wrote tests/golden/fullsize_digests.json (from the oracle alone); its digest
    functions are reused so that both sides hash the same bytes."""
    spec = importlib.util.spec_from_file_location("make_fullsize_golden", os.path.join(GOLDEN, "make_fullsize_golden.py"))
    mod = importlib.util.module_from_spec(spec)
    spec.loader.exec_module(mod)
    return mod

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


def run_full(rcd, wl, **cfg):
    import torch
    dev = torch.device("cuda", 0)
    with rcd.Context(0, **cfg) as ctx:
        X = rcd.features_to_torch(wl.features, device=dev)
        y = torch.from_numpy(wl.labels).to(dev)
        M = wl.N // wl.L
        a, o, v = ctx.rcd_partition(X, y, wl.capacities, wl.L, M_max=M)
        vals, total = ctx.rcd_objective(X, y, a, wl.W, wl.L, M_max=M)
        ctx.sync_status()
        return a.cpu().numpy(), o.cpu().numpy(), v.cpu().numpy(), vals.cpu().numpy()


def check_invariants(orc, wl, a, o):
    assert a.min() >= 0 and a.max() < wl.W
    assert np.array_equal(np.sort(o), np.arange(wl.N))               # every sample picked exactly once
    groups = orc.split_by_label(wl.labels, wl.L)
    off = 0
    for l, ids in enumerate(groups):
        q = orc.quotas(len(ids), wl.capacities)
        assert np.array_equal(np.bincount(a[ids], minlength=wl.W), q), "class %d" % l
        assert set(o[off:off + len(ids)].tolist()) == set(ids.tolist())
        off += len(ids)
    return groups


def test_c2_full_size_int8(rcd, orc):
    from paper_2211_00839_b200.workloads import make_workload
    wl = make_workload("C2")
    a, o, v, recomputed = run_full(rcd, wl)
    groups = check_invariants(orc, wl, a, o)
    assert np.array_equal(v, recomputed)                              # tracked f == f from the definition (GPU)
    # one class against the oracle: final block values from the plain definition, a replayed prefix
    # of its picks, and one late pick (block 0's last sample) from the plain gains
    l = 3
    ids = groups[l]
    M = len(ids)
    S = orc.similarity(wl.features[ids])
    local_assign = a[ids]
    for j in range(wl.W):
        assert orc.f_plain(S, np.nonzero(local_assign == j)[0]) == v[l, j]
    q = orc.quotas(M, wl.capacities)
    picked = o[l * M:(l + 1) * M]
    local = np.searchsorted(ids, picked).astype(np.int32)
    blocks = a[picked]
    bad, stats, _ = orc.replay_class(S, q, blocks[:100], local[:100], 0.0)
    assert bad == -1 and stats[0] == 0 and stats[1] == 0
    t_last = int(np.nonzero(blocks == 0)[0][-1])                      # step at which block 0 was filled
    members = local[:t_last][blocks[:t_last] == 0]
    gains = orc.gains_plain(S, members)
    unassigned = np.ones(M, dtype=bool)
    unassigned[local[:t_last]] = False
    cand = np.nonzero(unassigned)[0]
    best = cand[np.argmax(gains[cand])]                               # argmax returns the lowest index among ties
    assert best == local[t_last]


def test_c3_full_size_bf16(rcd, orc):
    from paper_2211_00839_b200.workloads import make_workload
    wl = make_workload("C3")
    a, o, v, recomputed = run_full(rcd, wl)
    groups = check_invariants(orc, wl, a, o)
    assert np.allclose(v, recomputed, rtol=OBJ_RTOL)
    l = 7
    ids = groups[l]
    M = len(ids)
    S = orc.similarity(wl.features[ids])
    local_assign = a[ids]
    want = np.array([orc.f_plain(S, np.nonzero(local_assign == j)[0]) for j in range(wl.W)])
    assert np.allclose(v[l], want, rtol=OBJ_RTOL)
    q = orc.quotas(M, wl.capacities)
    picked = o[l * M:(l + 1) * M]
    local = np.searchsorted(ids, picked).astype(np.int32)
    bad, stats, _ = orc.replay_class(S, q, a[picked][:120], local[:120], PICK_RTOL)
    assert bad == -1, stats


def test_c4_full_size_bf16(rcd, orc):
    from paper_2211_00839_b200.workloads import make_workload
    wl = make_workload("C4")
    a, o, v, recomputed = run_full(rcd, wl)
    groups = check_invariants(orc, wl, a, o)
    assert np.allclose(v, recomputed, rtol=OBJ_RTOL)
    M = wl.N // wl.L
    for l in (0, 17, 42, 63, 99):                                     # whole classes, teacher-forced
        ids = groups[l]
        S = orc.similarity(wl.features[ids])
        q = orc.quotas(M, wl.capacities)
        picked = o[l * M:(l + 1) * M]
        local = np.searchsorted(ids, picked).astype(np.int32)
        bad, stats, fv = orc.replay_class(S, q, a[picked], local, PICK_RTOL)
        assert bad == -1, (l, stats)
        assert np.allclose(v[l], fv, rtol=OBJ_RTOL, atol=1e-9)


def test_c5_many_classes_int8(rcd, orc):
    """ImageNet-shaped classes (M=1300, d=2048, W=64) with 200 of the 1000 classes: whole classes
    must equal the oracle's run of the class alone."""
    from paper_2211_00839_b200.workloads import make_workload
    wl = make_workload("C5", L=200)
    a, o, v, recomputed = run_full(rcd, wl)
    groups = check_invariants(orc, wl, a, o)
    assert np.array_equal(v, recomputed)
    M = wl.N // wl.L
    for l in (0, 77, 199):
        ids = groups[l]
        S = orc.similarity(wl.features[ids])
        q = orc.quotas(M, wl.capacities)
        assign, oj, ov, fv = orc.partition_class(S, q, "incremental")
        assert np.array_equal(a[ids], assign)
        assert np.array_equal(o[l * M:(l + 1) * M], ids[ov])
        assert np.array_equal(v[l], fv)


# ----------------------------------------------------------------------------- whole trajectories at full size

def _check_against_digests(rcd, orc, name, **cfg):
    """Every class of a full-size int8 configuration, bit for bit: block of every sample, pick order and
    block values must hash to the digest the oracle's own run of that class produced (stored under
    tests/golden by a script that calls only the oracle)."""
    from paper_2211_00839_b200.workloads import make_workload
    gm = _golden_module()
    gold = json.load(open(os.path.join(GOLDEN, "fullsize_digests.json")))[name]
    wl = make_workload(name)
    assert gm.input_digest(wl) == gold["inputs"], "the generator no longer produces the inputs the digests were written for"
    a, o, v, recomputed = run_full(rcd, wl, **cfg)
    groups = check_invariants(orc, wl, a, o)
    assert np.array_equal(v, recomputed)
    assert int(v.sum()) == gold["total_objective"]
    bad = []
    off = 0
    for l, ids in enumerate(groups):
        picked = o[off:off + len(ids)]
        off += len(ids)
        local = np.searchsorted(ids, picked).astype(np.int32)
        if gm.class_digest(a[ids], local, v[l]) != gold["class_digests"][l]:
            bad.append(l)
    if bad:                                                           # show where the first bad class leaves the oracle's path
        l = bad[0]
        ids = groups[l]
        S = orc.similarity(wl.features[ids])
        assign, oj, ov, fv = orc.partition_class(S, orc.quotas(len(ids), wl.capacities), "incremental")
        start = int(sum(len(g) for g in groups[:l]))
        local = np.searchsorted(ids, o[start:start + len(ids)])
        first = int(np.argmax(local != ov)) if np.any(local != ov) else -1
        pytest.fail("%s: %d classes differ from the oracle (first: class %d, first differing pick %d)" % (name, len(bad), l, first))


def test_c2_every_class_bit_exact(rcd, orc):
    """All 10 classes of C2 (5000 picks each) in the configuration bench.py times."""
    _check_against_digests(rcd, orc, "C2")


def test_c2_every_class_bit_exact_with_lazy_evaluation(rcd, orc):
    """The same 10 x 5000 picks with row-skipping passes switched on."""
    _check_against_digests(rcd, orc, "C2", lazy_mode=1, incremental=2)


def test_c2_every_class_bit_exact_without_incremental_updates(rcd, orc):
    """... and with every block waiting for a pass after each sample it receives (the bandwidth-bound form)."""
    _check_against_digests(rcd, orc, "C2", incremental=2)


def test_c5_every_class_bit_exact_with_incremental_updates(rcd, orc):
    """All 1000 classes with the in-place correction of stored gains forced on (the library leaves it off for this shape)."""
    _check_against_digests(rcd, orc, "C5", incremental=1)


def test_c5_every_class_bit_exact(rcd, orc):
    """All 1000 classes of C5 (1300 picks each)."""
    _check_against_digests(rcd, orc, "C5")


def test_c3_whole_classes_teacher_forced(rcd, orc):
    """Two whole classes of full-size C3 (5000 picks each, every one of them) replayed by the oracle in double:
    each pick's block within 1e-3 of the least value and its sample within 1e-3 of the best gain, tracked
    values within 1e-4 of the replayed ones.  The two replays run in two threads (the oracle is plain C)."""
    from paper_2211_00839_b200.workloads import make_workload
    wl = make_workload("C3")
    a, o, v, recomputed = run_full(rcd, wl)
    groups = check_invariants(orc, wl, a, o)
    M = wl.N // wl.L

    def replay(l):
        ids = groups[l]
        S = orc.similarity(wl.features[ids])
        q = orc.quotas(M, wl.capacities)
        picked = o[l * M:(l + 1) * M]
        local = np.searchsorted(ids, picked).astype(np.int32)
        return l, orc.replay_class(S, q, a[picked], local, PICK_RTOL)

    with ThreadPoolExecutor(max_workers=2) as ex:
        for l, (bad, stats, fv) in ex.map(replay, (2, 7)):
            print("C3 class %d: %d picks replayed, block mismatches %d (worst excess %.3g), sample mismatches %d (worst deficit %.3g)"
                  % (l, M, stats[0], stats[2], stats[1], stats[3]))
            assert bad == -1, (l, bad, stats)
            assert np.allclose(v[l], fv, rtol=OBJ_RTOL, atol=1e-9)
