"""Parity of the CUDA library (through its C ABI) against the CPU oracle, on the same seeded inputs.

int8 features: bit-exact (assignment, pick order, int64 objective).
bf16 features: objective within 1e-4 relative; picks equal to the oracle's wherever the
oracle's top-two candidates differ by more than 1e-3 relative (teacher-forced replay).
"""
import numpy as np
import pytest

pytestmark = pytest.mark.gpu

OBJ_RTOL = 1e-4      # final objective, float configs
PICK_RTOL = 1e-3     # a pick may differ from the oracle's only inside this relative gap
FREE_RUN_BRANCH_RTOL = 1e-4   # totals of two runs that took different branches at a near-tie (see check_float)


@pytest.fixture(scope="module")
def rcd():
    import torch
    assert torch.cuda.is_available()
    from paper_2211_00839_b200 import binding
    return binding


@pytest.fixture(scope="module")
def orc():
    from oracle import rcd_oracle
    return rcd_oracle


def to_device(rcd, wl):
    import torch
    dev = torch.device("cuda", 0)
    X = rcd.features_to_torch(wl.features, device=dev)
    y = torch.from_numpy(wl.labels).to(dev)
    return X, y


def run_partition(rcd, wl, **cfg):
    import torch
    with rcd.Context(0, **cfg) as ctx:
        X, y = to_device(rcd, wl)
        a, o, v = ctx.rcd_partition(X, y, wl.capacities, wl.L)
        ctx.sync_status()
        return a.cpu().numpy(), o.cpu().numpy(), v.cpu().numpy()


# ----------------------------------------------------------------------------- similarity

@pytest.mark.parametrize("M,d,batch", [(200, 64, 2), (257, 100, 1), (130, 37, 3), (1, 5, 1), (515, 512, 1)])
@pytest.mark.parametrize("path", [0, 2])
def test_similarity_int8_exact(rcd, orc, M, d, batch, path):
    import torch
    rng = np.random.default_rng(M * 1000 + d)
    X = rng.integers(-128, 128, size=(batch, M, d)).astype(np.int8)
    with rcd.Context(0, similarity_path=path) as ctx:
        S = ctx.rcd_similarity(torch.from_numpy(X).cuda())
        ctx.sync_status()
        # rows that are 16-byte multiples of at least 128 bytes must take the tensor-core kernel
        assert ctx.profile()["similarity_tc_launches"] == (1 if path == 0 and d % 16 == 0 and d >= 128 else 0)
        S = S.cpu().numpy()
    ld = (M + 3) // 4 * 4
    assert S.shape == (batch, M, ld)
    for b in range(batch):
        want = orc.similarity(X[b])
        assert np.array_equal(S[b, :, :M].astype(np.int64), want)
        assert np.all(S[b, :, M:] == 0)


@pytest.mark.parametrize("M,d,batch", [(200, 64, 2), (257, 104, 1), (131, 37, 2), (515, 2048, 1)])
@pytest.mark.parametrize("path", [0, 2])
def test_similarity_bf16_close(rcd, orc, M, d, batch, path):
    import torch
    from paper_2211_00839_b200.workloads import fp32_to_bf16_bits
    rng = np.random.default_rng(M * 7 + d)
    x = np.abs(rng.standard_normal((batch, M, d))).astype(np.float32)
    x /= np.linalg.norm(x, axis=2, keepdims=True)
    bits = fp32_to_bf16_bits(x)
    with rcd.Context(0, similarity_path=path) as ctx:
        S = ctx.rcd_similarity(rcd.features_to_torch(bits.reshape(batch * M, d)).view(batch, M, d).cuda())
        ctx.sync_status()
        assert ctx.profile()["similarity_tc_launches"] == (1 if path == 0 and (2 * d) % 16 == 0 and 2 * d >= 128 else 0)
        S = S.cpu().numpy()
    for b in range(batch):
        want = orc.similarity(bits[b])
        # fp32 accumulation of d products of magnitude <= 1/d-ish: absolute error far below 1e-5
        assert np.allclose(S[b, :, :M], want, rtol=2e-5, atol=2e-6)
        assert np.all(S[b, :, M:] == 0)


# ----------------------------------------------------------------------------- partition, int8: bit-exact

def check_exact(rcd, orc, wl, variant="incremental", **cfg):
    a, o, v = run_partition(rcd, wl, **cfg)
    ref = orc.partition(wl.features, wl.labels, wl.capacities, wl.L, variant=variant)
    assert np.array_equal(a, ref.assignment)
    assert np.array_equal(o, ref.order)
    assert np.array_equal(v, ref.part_values)
    return a, o, v, ref


@pytest.mark.parametrize("path", [0, 1, 2, 3, 4])  # chosen by the library / two launches per round / one launch with rounds / asynchronous / one CTA per class
@pytest.mark.parametrize("batch", [1, 2, 4, 8])
def test_partition_c1_exact(rcd, orc, batch, path):
    from paper_2211_00839_b200.workloads import make_workload
    wl = make_workload("C1")
    a, o, v, ref = check_exact(rcd, orc, wl, variant="plain", sweep_batch_max=batch, greedy_path=path)
    for l in range(wl.L):
        ids = np.nonzero(wl.labels == l)[0]
        assert np.bincount(a[ids], minlength=wl.W).tolist() == [25, 25, 50, 100]


@pytest.mark.parametrize("seed", [0, 1])
def test_partition_int8_ragged_classes(rcd, orc, seed):
    """Unequal class sizes (several tiles and a ragged tail), an empty class, a class smaller than W,
    a feature width that is not a multiple of 4."""
    from paper_2211_00839_b200.workloads import Workload, make_mixture
    rng = np.random.default_rng(40 + seed)
    sizes = [333, 0, 5, 1030, 1, 257]
    d = 75
    feats, labels = [], []
    for l, M in enumerate(sizes):
        x = make_mixture(rng, M, d, 4, "dirichlet", "gauss", 4.0) if M else np.zeros((0, d), np.float32)
        feats.append(np.clip(np.rint(x), -127, 127).astype(np.int8))
        labels.append(np.full(M, l, np.int32))
    feats = np.concatenate(feats)
    labels = np.concatenate(labels)
    perm = rng.permutation(len(labels))
    caps = np.array([1, 2.5, 1, 4, 0.5, 3, 1, 1, 2], dtype=np.float64)
    wl = Workload("ragged", "int8", np.ascontiguousarray(feats[perm]), np.ascontiguousarray(labels[perm]), caps,
                  len(sizes), len(caps))
    for batch, path in ((8, 0), (1, 0), (8, 1), (8, 2), (8, 3), (2, 3), (8, 4), (4, 4)):
        check_exact(rcd, orc, wl, sweep_batch_max=batch, greedy_path=path)


def test_partition_int8_ties_and_duplicates(rcd, orc):
    """Duplicate rows and one-hot rows: every argmax / argmin tie must fall to the lowest index."""
    from paper_2211_00839_b200.workloads import Workload
    rng = np.random.default_rng(3)
    base = rng.integers(-5, 6, size=(12, 16)).astype(np.int8)
    feats = np.concatenate([base[rng.integers(0, 12, size=90)], 9 * np.eye(30, 16, dtype=np.int8)])
    labels = np.concatenate([np.zeros(90, np.int32), np.ones(30, np.int32)])
    wl = Workload("ties", "int8", feats, labels, np.array([1.0, 1.0, 2.0]), 2, 3)
    check_exact(rcd, orc, wl, variant="plain")


def test_partition_c2_reduced_exact(rcd, orc):
    from paper_2211_00839_b200.workloads import make_workload
    wl = make_workload("C2", L=3, M=1200)
    check_exact(rcd, orc, wl)


def test_partition_c5_reduced_exact(rcd, orc):
    from paper_2211_00839_b200.workloads import make_workload
    wl = make_workload("C5", L=6, M=700, d=256)
    check_exact(rcd, orc, wl)


@pytest.mark.parametrize("path", [2, 3, 4])
def test_partition_many_small_classes_every_loop_form(rcd, orc, path):
    """More classes than pick CTAs of the asynchronous loop (a pick CTA then serves several classes), of
    unequal sizes so that classes finish at different times; W = 64 with threshold passes."""
    from paper_2211_00839_b200.workloads import Workload, make_workload
    base = make_workload("C5", L=60, M=160, d=128)
    rng = np.random.default_rng(7)
    keep = np.ones(base.N, bool)
    for l in range(base.L):                       # thin every class by a different amount
        ids = np.nonzero(base.labels == l)[0]
        keep[ids[:int(rng.integers(0, 100))]] = False
    wl = Workload("many", "int8", np.ascontiguousarray(base.features[keep]), np.ascontiguousarray(base.labels[keep]),
                  base.capacities, base.L, base.W)
    check_exact(rcd, orc, wl, greedy_path=path)


def test_partition_is_reproducible(rcd):
    from paper_2211_00839_b200.workloads import make_workload
    wl = make_workload("C3", L=2, M=600, d=128)
    r1 = run_partition(rcd, wl)
    r2 = run_partition(rcd, wl)
    for x, y in zip(r1, r2):
        assert np.array_equal(x, y)


def ragged_float_workload(sizes, d, W, seed):
    from paper_2211_00839_b200.workloads import Workload, make_mixture, fp32_to_bf16_bits
    rng = np.random.default_rng(seed)
    feats, labels = [], []
    for l, M in enumerate(sizes):
        x = make_mixture(rng, M, d, 4, "dirichlet", "gauss", 4.0) if M else np.zeros((0, d), np.float32)
        x = x / np.maximum(np.linalg.norm(x, axis=1, keepdims=True), 1e-30)
        feats.append(fp32_to_bf16_bits(x.astype(np.float32)))
        labels.append(np.full(M, l, np.int32))
    feats = np.concatenate(feats)
    labels = np.concatenate(labels)
    perm = rng.permutation(len(labels))
    caps = rng.uniform(1.0, 4.0, size=W)
    return Workload("ragged-float", "bf16", np.ascontiguousarray(feats[perm]), np.ascontiguousarray(labels[perm]), caps,
                    len(sizes), W)


@pytest.mark.parametrize("path", [2, 3, 4])
def test_float_partition_is_reproducible_with_ragged_classes(rcd, path):
    """fp32 gains depend on how a pass splits its columns, so the shape of a class's sweeps must not depend on
    when OTHER classes finish: classes of very unequal sizes (the small ones finish while the large ones
    run), both one-launch forms of the loop, several runs, bit-identical outputs."""
    wl = ragged_float_workload([1500, 40, 700, 9, 260, 1100, 130], d=128, W=12, seed=91)
    first = run_partition(rcd, wl, greedy_path=path)
    for _ in range(4):
        again = run_partition(rcd, wl, greedy_path=path)
        for x, y in zip(first, again):
            assert np.array_equal(x, y)


@pytest.mark.parametrize("name,kw,W", [("C2", dict(L=3, M=1003), 7), ("C1", {}, 3)])
def test_equal_capacities_is_the_label_balanced_partition(rcd, orc, name, kw, W):
    """Algorithm 3 (all ratios equal): block sizes inside a class differ by at most one, and the result is the
    oracle's, bit for bit."""
    from paper_2211_00839_b200.workloads import Workload, make_workload
    base = make_workload(name, **kw)
    wl = Workload("equal", base.dtype, base.features, base.labels, np.full(W, 2.5), base.L, W)
    a, o, v, ref = check_exact(rcd, orc, wl)
    for l in range(wl.L):
        sizes = np.bincount(a[wl.labels == l], minlength=W)
        assert sizes.max() - sizes.min() <= 1 and sizes.sum() == np.count_nonzero(wl.labels == l)


# ----------------------------------------------------------------------------- partition, bf16: tolerance rule

def check_float(rcd, orc, wl, **cfg):
    a, o, v = run_partition(rcd, wl, **cfg)
    free = orc.partition(wl.features, wl.labels, wl.capacities, wl.L, variant="incremental")
    groups = orc.split_by_label(wl.labels, wl.L)
    total_replayed = 0.0
    same_everywhere = True
    for l, ids in enumerate(groups):
        M = len(ids)
        if M == 0:
            continue
        q = orc.quotas(M, wl.capacities)
        assert np.bincount(a[ids], minlength=wl.W).tolist() == q.tolist()
        off = int(free.class_offsets[l])
        picked = o[off:off + M]
        assert sorted(picked.tolist()) == sorted(ids.tolist())
        local = np.searchsorted(ids, picked).astype(np.int32)
        S = orc.similarity(wl.features[ids])
        bad, stats, fv = orc.replay_class(S, q, a[picked], local, PICK_RTOL)
        assert bad == -1, "class %d: pick %d outside the %g gap (stats %s)" % (l, bad, PICK_RTOL, stats)
        # tracked (fp32 gains summed in fp64) vs the oracle's value of the same picks
        assert np.allclose(v[l], fv, rtol=OBJ_RTOL, atol=1e-9)
        total_replayed += fv.sum()
        # free-running oracle: identical picks up to the first step whose top-two gap is inside the tolerance
        ref_picked = free.order[off:off + M]
        same = (picked == ref_picked) & (a[picked] == free.order_block[off:off + M])
        if not same.all():
            same_everywhere = False
            first = int(np.argmin(same))
            bad0, stats0, _ = orc.replay_class(S, q, a[picked][:first + 1], local[:first + 1], 0.0)
            assert bad0 == first and max(stats0[2], stats0[3]) <= PICK_RTOL
    assert abs(v.sum() - total_replayed) <= OBJ_RTOL * abs(total_replayed)
    # The free-running oracle: while every pick is the same, its total must agree to OBJ_RTOL as well.  Once a
    # pick inside the 1e-3 gap has gone the other way the two runs are different (both valid) trajectories; on the
    # synthetic workloads their totals still agree to OBJ_RTOL (measured: below 1e-6), which is what is asserted.
    free_dev = abs(v.sum() - free.total) / abs(free.total)
    print("free-run deviation %.3g (%s), replayed deviation %.3g" % (
        free_dev, "same picks" if same_everywhere else "a near-tie went the other way",
        abs(v.sum() - total_replayed) / abs(total_replayed)))
    assert free_dev <= (OBJ_RTOL if same_everywhere else FREE_RUN_BRANCH_RTOL)
    return a, o, v


def test_partition_c3_reduced_float(rcd, orc):
    from paper_2211_00839_b200.workloads import make_workload
    wl = make_workload("C3", L=2, M=900, d=512)
    check_float(rcd, orc, wl)


@pytest.mark.parametrize("batch,path", [(1, 0), (8, 0), (8, 1), (8, 2), (8, 3), (8, 4)])
def test_partition_c4_reduced_float(rcd, orc, batch, path):
    from paper_2211_00839_b200.workloads import make_workload
    wl = make_workload("C4", L=5, M=500, d=256)
    check_float(rcd, orc, wl, sweep_batch_max=batch, greedy_path=path)


# ----------------------------------------------------------------------------- threshold passes

def run_with_profile(rcd, wl, **cfg):
    with rcd.Context(0, profile=1, **cfg) as ctx:
        X, y = to_device(rcd, wl)
        a, o, v = ctx.rcd_partition(X, y, wl.capacities, wl.L)
        ctx.sync_status()
        return a.cpu().numpy(), o.cpu().numpy(), v.cpu().numpy(), ctx.profile()


@pytest.mark.parametrize("path", [0, 1, 2, 3, 4])
def test_threshold_passes_int8_exact(rcd, orc, path):
    """Classes large enough that the sweeps switch to threshold passes: same picks as the oracle, and
    the same as with dense passes only."""
    from paper_2211_00839_b200.workloads import make_workload
    wl = make_workload("C2", L=3, M=1200)
    ref = orc.partition(wl.features, wl.labels, wl.capacities, wl.L, variant="incremental")
    # (incremental = 2: every block that received a sample waits for a pass, so that threshold passes are what runs)
    a, o, v, prof = run_with_profile(rcd, wl, greedy_path=path, incremental=2)
    assert prof["threshold_elems"] > 0 and 0 < prof["threshold_hits"] < prof["threshold_elems"] // 32
    assert np.array_equal(a, ref.assignment) and np.array_equal(o, ref.order) and np.array_equal(v, ref.part_values)
    a1, o1, v1, prof1 = run_with_profile(rcd, wl, greedy_path=path, sweep_mode=1, incremental=2)
    assert prof1["threshold_elems"] == 0
    assert np.array_equal(a1, a) and np.array_equal(o1, o) and np.array_equal(v1, v)


@pytest.mark.parametrize("knobs", [dict(greedy_path=3, async_group=1), dict(greedy_path=3, async_group=2, async_help_min=1),
                                   dict(greedy_path=3, async_help_min=400), dict(threshold_from=1), dict(threshold_from=2, threshold_hit_shift=3),
                                   dict(greedy_path=2, threshold_from=1, threshold_hit_shift=7), dict(greedy_path=1, threshold_from=3),
                                   dict(greedy_path=4, threshold_from=2, sweep_batch_max=4)])
def test_scheduling_knobs_never_change_a_result(rcd, orc, knobs):
    """Serving order of the asynchronous loop and the start / back-off rule of the threshold passes only move
    work around: assignment, pick order and block values stay those of the oracle."""
    from paper_2211_00839_b200.workloads import make_workload
    wl = make_workload("C2", L=4, M=900)
    check_exact(rcd, orc, wl, **knobs)


def test_threshold_passes_many_blocks_exact(rcd, orc):
    """W = 64: one threshold pass refreshes more than 32 blocks (two blocks per lane)."""
    from paper_2211_00839_b200.workloads import make_workload
    wl = make_workload("C5", L=3, M=1300, d=128)
    ref = orc.partition(wl.features, wl.labels, wl.capacities, wl.L, variant="incremental")
    a, o, v, prof = run_with_profile(rcd, wl, incremental=2)
    assert prof["threshold_elems"] > 0 and prof["threshold_max_blocks"] > 32
    assert np.array_equal(a, ref.assignment) and np.array_equal(o, ref.order) and np.array_equal(v, ref.part_values)


def test_threshold_passes_float(rcd, orc):
    from paper_2211_00839_b200.workloads import make_workload
    wl = make_workload("C3", L=2, M=900, d=512)
    with rcd.Context(0, profile=1, incremental=2) as ctx:
        X, y = to_device(rcd, wl)
        ctx.rcd_partition(X, y, wl.capacities, wl.L)
        ctx.sync_status()
        assert ctx.profile()["threshold_elems"] > 0
    check_float(rcd, orc, wl, incremental=2)        # the run above
    check_float(rcd, orc, wl, sweep_mode=1, incremental=2)


# ----------------------------------------------------------------------------- incremental update of stored gains

@pytest.mark.parametrize("path", [3, 4])
def test_incremental_update_int8_exact(rcd, orc, path):
    """A pick that raises its block's coverage in few columns corrects the block's stored gains in place (one row of S
    per column); the block then needs no pass.  Same picks as the oracle, and as with the correction switched off."""
    from paper_2211_00839_b200.workloads import make_workload
    wl = make_workload("C2", L=3, M=1200)
    ref = orc.partition(wl.features, wl.labels, wl.capacities, wl.L, variant="incremental")
    a, o, v, prof = run_with_profile(rcd, wl, greedy_path=path, incremental=1)
    assert prof["incremental_updates"] > 1000 and prof["incremental_rows"] >= prof["incremental_updates"] // 2
    assert prof["noted_picks"] > prof["incremental_updates"] // 2      # most picks take v* from the note of the last correction
    assert np.array_equal(a, ref.assignment) and np.array_equal(o, ref.order) and np.array_equal(v, ref.part_values)
    a0, o0, v0, prof0 = run_with_profile(rcd, wl, greedy_path=path, incremental=2)
    assert prof0["incremental_updates"] == 0
    assert np.array_equal(a0, a) and np.array_equal(o0, o) and np.array_equal(v0, v)
    assert prof["sweep_bytes"] < prof0["sweep_bytes"]


def test_incremental_update_many_blocks_ragged_ties_exact(rcd, orc):
    """W = 64 with short rows (twelve rows of S in flight per thread), ragged classes with duplicate rows (ties), several
    caps on the number of raised columns, both loop forms that carry the correction."""
    from paper_2211_00839_b200.workloads import Workload, make_workload
    wl = make_workload("C5", L=3, M=1300, d=128)
    for path, cap in ((4, 0), (4, 5), (3, 0), (3, 128)):
        check_exact(rcd, orc, wl, greedy_path=path, incremental=1, incremental_max=cap)
    base = make_workload("C2", L=40, M=300, d=64)
    rng = np.random.default_rng(29)
    keep = np.ones(base.N, bool)
    for l in range(base.L):
        ids = np.nonzero(base.labels == l)[0]
        keep[ids[:int(rng.integers(0, 200))]] = False
    feats = base.features[keep].copy()
    feats[::7] = feats[3]
    wl2 = Workload("ragged-inc", "int8", np.ascontiguousarray(feats), np.ascontiguousarray(base.labels[keep]), base.capacities, base.L, base.W)
    for path in (3, 4):
        check_exact(rcd, orc, wl2, greedy_path=path, incremental=1)


@pytest.mark.parametrize("path", [3, 4])
def test_incremental_update_float(rcd, orc, path):
    from paper_2211_00839_b200.workloads import make_workload
    wl = make_workload("C3", L=2, M=900, d=512)
    with rcd.Context(0, profile=1, greedy_path=path, incremental=1) as ctx:
        X, y = to_device(rcd, wl)
        ctx.rcd_partition(X, y, wl.capacities, wl.L)
        ctx.sync_status()
        assert ctx.profile()["incremental_updates"] > 0
    check_float(rcd, orc, wl, greedy_path=path, incremental=1)
    check_float(rcd, orc, wl, greedy_path=path, incremental=1, incremental_max=4)
    r1 = run_partition(rcd, wl, greedy_path=path, incremental=1)
    r2 = run_partition(rcd, wl, greedy_path=path, incremental=1)
    for x, y in zip(r1, r2):
        assert np.array_equal(x, y)                      # the corrections are applied in a fixed order


@pytest.mark.parametrize("path", [3, 4])
def test_noted_candidates_ties_and_many_classes(rcd, orc, path):
    """Picks that take v* from the note made at the block's last correction (up to sixteen blocks per class keep notes): duplicate samples
    make equal gains (the lowest index must win, also when the noted sample of one block is taken by another block first),
    ragged classes, more classes than SMs in the one-CTA-per-class form; twice, with identical results."""
    from paper_2211_00839_b200.workloads import Workload, make_workload
    L = 12 if path == 3 else 200
    base = make_workload("C2", L=L, M=260, d=64, seed=77)
    rng = np.random.default_rng(31)
    keep = np.ones(base.N, bool)
    for l in range(base.L):
        ids = np.nonzero(base.labels == l)[0]
        keep[ids[:int(rng.integers(0, 120))]] = False
    feats = base.features[keep].copy()
    feats[::5] = feats[2]                                # a fifth of all samples are copies of one: ties everywhere
    feats[1::11] = feats[4]
    wl = Workload("noted", "int8", np.ascontiguousarray(feats), np.ascontiguousarray(base.labels[keep]), base.capacities, base.L, base.W)
    ref = orc.partition(wl.features, wl.labels, wl.capacities, wl.L, variant="incremental")
    a, o, v, prof = run_with_profile(rcd, wl, greedy_path=path, incremental=1)
    assert prof["noted_picks"] > 0
    assert np.array_equal(a, ref.assignment) and np.array_equal(o, ref.order) and np.array_equal(v, ref.part_values)
    a2, o2, v2, prof2 = run_with_profile(rcd, wl, greedy_path=path, incremental=1)
    assert np.array_equal(a2, a) and np.array_equal(o2, o) and np.array_equal(v2, v) and prof2["noted_picks"] == prof["noted_picks"]


# ----------------------------------------------------------------------------- exact lazy evaluation (row-skipping passes)

@pytest.mark.parametrize("path", [0, 1, 2, 3, 4])
def test_lazy_evaluation_int8_exact(rcd, orc, path):
    """Row-skipping threshold passes (stored gains as upper bounds, a floor per block): rows are skipped, some picks
    miss and are answered by a pass over every row, and every pick is still the oracle's."""
    from paper_2211_00839_b200.workloads import make_workload
    wl = make_workload("C2", L=3, M=1200)
    ref = orc.partition(wl.features, wl.labels, wl.capacities, wl.L, variant="incremental")
    a, o, v, prof = run_with_profile(rcd, wl, greedy_path=path, lazy_mode=1, lazy_from=2, incremental=2)
    assert prof["lazy_sweeps"] > 0 and prof["lazy_rows_skipped"] > prof["lazy_rows"] > 0 and prof["lazy_misses"] > 0
    assert np.array_equal(a, ref.assignment) and np.array_equal(o, ref.order) and np.array_equal(v, ref.part_values)
    a0, o0, v0, prof0 = run_with_profile(rcd, wl, greedy_path=path, incremental=2)
    assert prof0["lazy_sweeps"] == 0 and prof0["lazy_rows"] == 0
    assert prof["sweep_bytes"] < prof0["sweep_bytes"]


@pytest.mark.parametrize("lazy_from", [1, 8])
def test_lazy_evaluation_many_blocks_and_ragged_classes_exact(rcd, orc, lazy_from):
    """W = 64 (two blocks per lane in a pass), classes of unequal sizes, more classes than pick CTAs."""
    from paper_2211_00839_b200.workloads import Workload, make_workload
    wl = make_workload("C5", L=3, M=1300, d=128)
    ref = orc.partition(wl.features, wl.labels, wl.capacities, wl.L, variant="incremental")
    a, o, v, prof = run_with_profile(rcd, wl, lazy_mode=1, lazy_from=lazy_from, incremental=2)
    assert prof["lazy_sweeps"] > 0
    assert np.array_equal(a, ref.assignment) and np.array_equal(o, ref.order) and np.array_equal(v, ref.part_values)
    base = make_workload("C2", L=40, M=300, d=64)
    rng = np.random.default_rng(17)
    keep = np.ones(base.N, bool)
    for l in range(base.L):
        ids = np.nonzero(base.labels == l)[0]
        keep[ids[:int(rng.integers(0, 200))]] = False
    wl = Workload("ragged-lazy", "int8", np.ascontiguousarray(base.features[keep]), np.ascontiguousarray(base.labels[keep]),
                  base.capacities, base.L, base.W)
    for path in (2, 3, 4):
        check_exact(rcd, orc, wl, greedy_path=path, lazy_mode=1, lazy_from=lazy_from, incremental=2)


def test_lazy_evaluation_float(rcd, orc):
    from paper_2211_00839_b200.workloads import make_workload
    wl = make_workload("C3", L=2, M=900, d=512)
    with rcd.Context(0, profile=1, lazy_mode=1, lazy_from=2, incremental=2) as ctx:
        X, y = to_device(rcd, wl)
        ctx.rcd_partition(X, y, wl.capacities, wl.L)
        ctx.sync_status()
        assert ctx.profile()["lazy_sweeps"] > 0
    check_float(rcd, orc, wl, lazy_mode=1, lazy_from=2, incremental=2)
    check_float(rcd, orc, wl, lazy_mode=1, greedy_path=2)


# ----------------------------------------------------------------------------- objective

@pytest.mark.parametrize("name,L,M,d", [("C1", 2, 200, 64), ("C5", 3, 300, 128), ("C4", 3, 250, 96)])
def test_objective_matches_plain_definition(rcd, orc, name, L, M, d):
    import torch
    from paper_2211_00839_b200.workloads import make_workload
    wl = make_workload(name, L=L, M=M, d=d)
    rng = np.random.default_rng(5)
    assignment = rng.integers(-1, wl.W, size=wl.N).astype(np.int32)     # arbitrary, -1 = in no block
    with rcd.Context(0) as ctx:
        X, y = to_device(rcd, wl)
        vals, total = ctx.rcd_objective(X, y, torch.from_numpy(assignment).cuda(), wl.W, wl.L)
        ctx.sync_status()
        vals, total = vals.cpu().numpy(), total.cpu().numpy()
    want = orc.objective(wl.features, wl.labels, assignment, wl.W, wl.L)
    if wl.dtype == "int8":
        assert np.array_equal(vals, want) and total[0] == want.sum()
    else:
        assert np.allclose(vals, want, rtol=1e-5, atol=1e-7)
        assert total[0] == pytest.approx(want.sum(), rel=1e-5)


def test_tracked_values_equal_recomputed_objective(rcd):
    import torch
    from paper_2211_00839_b200.workloads import make_workload
    wl = make_workload("C2", L=2, M=800)
    with rcd.Context(0) as ctx:
        X, y = to_device(rcd, wl)
        a, o, v = ctx.rcd_partition(X, y, wl.capacities, wl.L)
        vals, total = ctx.rcd_objective(X, y, a, wl.W, wl.L)
        ctx.sync_status()
        assert torch.equal(v, vals) and int(total[0]) == int(v.sum())


# ----------------------------------------------------------------------------- host-buffer entry point, errors

def test_partition_host_matches_device_entry(rcd, orc):
    import torch
    from paper_2211_00839_b200.workloads import make_workload
    wl = make_workload("C1")
    ref = orc.partition(wl.features, wl.labels, wl.capacities, wl.L, variant="plain")
    with rcd.Context(0) as ctx:
        X = rcd.features_to_torch(wl.features, pin=True)
        y = torch.from_numpy(wl.labels).pin_memory()
        a, o, v = ctx.rcd_partition_host(X, y, wl.capacities, wl.L)
        assert np.array_equal(a.numpy(), ref.assignment)
        assert np.array_equal(o.numpy(), ref.order)
        assert np.array_equal(v.numpy(), ref.part_values)


def test_argument_errors_are_reported(rcd):
    import torch
    from paper_2211_00839_b200.workloads import make_workload
    wl = make_workload("C1")
    with rcd.Context(0) as ctx:
        X, y = to_device(rcd, wl)
        with pytest.raises(rcd.RcdError) as e:
            ctx.rcd_partition(X, y, [1.0, -1.0], wl.L)
        assert e.value.status == 1
        with pytest.raises(rcd.RcdError) as e:
            ctx.rcd_partition(X, y, [1.0, float("nan")], wl.L)
        assert e.value.status == 1
        with pytest.raises(rcd.RcdError) as e:       # a label outside [0, L)
            ctx.rcd_partition(X, y, wl.capacities, 1)
        assert e.value.status == 1
        with pytest.raises(rcd.RcdError) as e:       # class larger than promised -> workspace too small
            ctx._ws = None
            ctx.rcd_partition(X, y, wl.capacities, wl.L, M_max=10)
        assert e.value.status == 3
        # and the context still works afterwards
        a, o, v = ctx.rcd_partition(X, y, wl.capacities, wl.L)
        ctx.sync_status()
        assert int(a.min()) >= 0 and int(a.max()) < wl.W


def test_empty_input(rcd):
    import torch
    with rcd.Context(0) as ctx:
        X = torch.empty((0, 16), dtype=torch.int8, device="cuda")
        y = torch.empty((0,), dtype=torch.int32, device="cuda")
        a, o, v = ctx.rcd_partition(X, y, [1.0, 2.0], 3)
        ctx.sync_status()
        assert a.numel() == 0 and v.shape == (3, 2) and int(v.abs().sum()) == 0


def test_bounded_wait_times_out_as_a_status_not_a_hang(rcd):
    """A device-side wait that nothing can satisfy ends after its poll limit and surfaces as
    RCD_ERR_TIMEOUT; the context and the GPU stay usable."""
    import torch
    from paper_2211_00839_b200.workloads import make_workload
    wl = make_workload("C1")
    with rcd.Context(0) as ctx:
        ctx.selftest_bounded_wait()
        with pytest.raises(rcd.RcdError) as e:
            ctx.sync_status()
        assert e.value.status == 5          # RCD_ERR_TIMEOUT
        X, y = to_device(rcd, wl)
        a, o, v = ctx.rcd_partition(X, y, wl.capacities, wl.L)
        ctx.sync_status()                   # clean again
        assert int(a.min()) >= 0
