"""Pins for the CPU oracle: what the paper and the mathematics fix, independent of the oracle itself.

Each test names the passage it rests on.  None of these needs a GPU.
"""
import itertools
import json
import math
import os

import numpy as np
import pytest

from oracle import rcd_oracle as orc

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def rand_sym_int(rng, M, lo=-20, hi=60):
    A = rng.integers(lo, hi, size=(M, M))
    S = np.triu(A) + np.triu(A, 1).T
    return S.astype(np.int64)


def brute_f(S, A):
    """Facility location on a Python set, via numpy row maxima."""
    if len(A) == 0:
        return S.dtype.type(0)
    return np.maximum(S[:, sorted(A)].max(axis=1), 0).sum()


# ----------------------------------------------------------------------------- quotas (Algorithm 1, C_{l,j})

def test_quotas_worked_values():
    # 200 * (1,1,2,4)/8: exact shares
    assert orc.quotas(200, [1, 1, 2, 4]).tolist() == [25, 25, 50, 100]
    # 5000 * r/16: shares 312.5 x4, 625 x2, 1250 x2; two left-over units go to the lowest-index halves
    assert orc.quotas(5000, [1, 1, 1, 1, 2, 2, 4, 4]).tolist() == [313, 313, 312, 312, 625, 625, 1250, 1250]
    # 1300 over four tiers 1:2:4:8 of 16 workers: shares 5.4167, 10.8333, 21.6667, 43.3333 ->
    # floors sum to 1264, 36 left: 16 to tier 2 (.8333), 16 to tier 4 (.6667), 4 to the first tier-1 workers
    caps = [2.0 ** (j // 16) for j in range(64)]
    want = [6] * 4 + [5] * 12 + [11] * 16 + [22] * 16 + [43] * 16
    assert orc.quotas(1300, caps).tolist() == want


def test_quotas_sum_and_proportion():
    rng = np.random.default_rng(5)
    for _ in range(200):
        W = int(rng.integers(1, 40))
        M = int(rng.integers(0, 3000))
        r = rng.uniform(0.1, 9.0, size=W)
        q = orc.quotas(M, r)
        assert q.sum() == M                       # sum_j C_{l,j} = M  (Section 3.1 problem statement)
        ideal = M * r / r.sum()
        assert np.all(np.abs(q - ideal) < 1.0)    # each quota is the floor or the ceiling of its share
        assert np.all(q >= 0)


def test_quotas_equal_capacities_is_label_balanced():
    # Algorithm 3: C_l = |V_l| / N
    q = orc.quotas(103, [2.5] * 10)
    assert q.sum() == 103 and q.max() - q.min() <= 1
    assert q.tolist() == [11, 11, 11] + [10] * 7   # left-over units to the lowest indices


# ----------------------------------------------------------------------------- similarity

def test_similarity_int8_matches_integer_matmul():
    rng = np.random.default_rng(1)
    X = rng.integers(-128, 128, size=(37, 53)).astype(np.int8)
    S = orc.similarity(X)
    assert S.dtype == np.int64
    assert np.array_equal(S, X.astype(np.int64) @ X.astype(np.int64).T)


def test_similarity_bf16_is_dot_of_the_rounded_values():
    from paper_2211_00839_b200.workloads import fp32_to_bf16_bits, bf16_bits_to_fp32
    rng = np.random.default_rng(2)
    x = rng.standard_normal((19, 40)).astype(np.float32)
    bits = fp32_to_bf16_bits(x)
    S = orc.similarity(bits)
    xd = bf16_bits_to_fp32(bits).astype(np.float64)
    assert np.allclose(S, xd @ xd.T, rtol=1e-13, atol=1e-13)
    # one-hot rows: exact identity
    eye = fp32_to_bf16_bits(np.eye(5, 8, dtype=np.float32))
    assert np.array_equal(orc.similarity(eye), np.eye(5))


# ----------------------------------------------------------------------------- objective (Section 4 item 2)

def test_f_closed_forms():
    c = 7
    S = (c * np.eye(6)).astype(np.int64)
    for n in range(7):
        assert orc.f_plain(S, list(range(n))) == c * n          # S = cI: every member covers itself only
    S = np.full((5, 5), 3, dtype=np.int64)
    assert orc.f_plain(S, []) == 0                               # f(empty) = 0
    assert orc.f_plain(S, [2]) == 15 and orc.f_plain(S, [0, 4]) == 15
    S = -np.ones((4, 4), dtype=np.int64)
    assert orc.f_plain(S, [0, 1]) == 0                           # negative similarities are clamped
    S = np.array([[1.5, -2.0], [0.25, 4.0]])
    assert orc.f_plain(S, [0]) == 1.75 and orc.f_plain(S, [1]) == 4.0 and orc.f_plain(S, [0, 1]) == 5.5


def test_f_uses_rows_as_covered_points_and_columns_as_members():
    # non-symmetric S exposes a transposed operand: f(A) = sum_i max_{v' in A} S[i][v']
    S = np.array([[1, 9, 0], [2, 0, 0], [3, 0, 5]], dtype=np.int64)
    assert orc.f_plain(S, [0]) == 6          # column 0: 1+2+3
    assert orc.f_plain(S, [1]) == 9
    assert orc.f_plain(S, [0, 2]) == 1 + 2 + 5


def test_f_monotone_and_submodular_exhaustive():
    # Section 3.1: f(A u v) - f(A) >= 0, and diminishing returns for A subset B
    rng = np.random.default_rng(3)
    M = 6
    S = rand_sym_int(rng, M)
    subsets = [tuple(c) for k in range(M + 1) for c in itertools.combinations(range(M), k)]
    fval = {A: orc.f_plain(S, list(A)) for A in subsets}
    for A in subsets:
        assert fval[A] == brute_f(S, A)
    for B in subsets:
        for k in range(len(B) + 1):
            for A in itertools.combinations(B, k):
                for v in range(M):
                    if v in B:
                        continue
                    gA = fval[tuple(sorted(A + (v,)))] - fval[A]
                    gB = fval[tuple(sorted(B + (v,)))] - fval[B]
                    assert gB >= 0 and gA >= gB


def test_gains_plain_match_definition():
    rng = np.random.default_rng(4)
    S = rand_sym_int(rng, 9)
    A = [1, 4, 7]
    g = orc.gains_plain(S, A)
    for v in range(9):
        assert g[v] == brute_f(S, set(A) | {v}) - brute_f(S, set(A))


# ----------------------------------------------------------------------------- Algorithm 1: hand traces

@pytest.mark.parametrize("variant", ["plain", "incremental"])
@pytest.mark.parametrize("as_float", [False, True])
def test_hand_worked_traces(variant, as_float):
    cases = json.load(open(os.path.join(GOLDEN, "hand_traces.json")))["cases"]
    for c in cases:
        S = np.array(c["S"], dtype=np.float64 if as_float else np.int64)
        assign, oj, ov, fv = orc.partition_class(S, c["quotas"], variant, objective=c.get("objective", "facility"))
        assert oj.tolist() == c["order_j"], c["name"]
        assert ov.tolist() == c["order_v"], c["name"]
        assert assign.tolist() == c["assign"], c["name"]
        assert fv.tolist() == c["fvals"], c["name"]


# ----------------------------------------------------------------------------- special cases that reduce to tie-break order

def round_robin_by_count(M, quotas, c):
    """S = cI: every gain is c, f_j = c*|A_j|; so the block is the least-filled non-full one
    (lowest index on ties) and the sample is the lowest unassigned index."""
    cnt = [0] * len(quotas)
    assign = [-1] * M
    for v in range(M):
        open_blocks = [j for j in range(len(quotas)) if cnt[j] < quotas[j]]
        j = min(open_blocks, key=lambda p: (cnt[p], p))
        assign[v] = j
        cnt[j] += 1
    return assign


@pytest.mark.parametrize("variant", ["plain", "incremental"])
def test_scaled_identity_is_round_robin(variant):
    M, caps = 23, [1, 2, 3.5]
    q = orc.quotas(M, caps)
    S = (11 * np.eye(M)).astype(np.int64)
    assign, oj, ov, fv = orc.partition_class(S, q, variant)
    assert ov.tolist() == list(range(M))
    assert assign.tolist() == round_robin_by_count(M, q.tolist(), 11)
    assert fv.tolist() == (11 * q).tolist()


@pytest.mark.parametrize("variant", ["plain", "incremental"])
def test_identical_rows_fill_blocks_in_index_order(variant):
    # all similarities equal c>0: a block's first member covers everything (gain M*c), later gains are 0.
    # So blocks 0..W-1 take samples 0..W-1, then all f are equal and the lowest non-full block is filled up.
    M, q = 12, [3, 5, 4]
    S = np.full((M, M), 2, dtype=np.int64)
    assign, oj, ov, fv = orc.partition_class(S, q, variant)
    assert ov.tolist() == list(range(M))
    assert oj.tolist() == [0, 1, 2] + [0] * 2 + [1] * 4 + [2] * 3
    assert fv.tolist() == [2 * M] * 3


def test_single_block_takes_everything():
    from paper_2211_00839_b200.workloads import fp32_to_bf16_bits
    rng = np.random.default_rng(6)
    x = rng.standard_normal((30, 16)).astype(np.float32)
    x /= np.linalg.norm(x, axis=1, keepdims=True)
    S = orc.similarity(fp32_to_bf16_bits(x))
    assign, oj, ov, fv = orc.partition_class(S, [30], "plain")
    assert assign.tolist() == [0] * 30 and sorted(ov.tolist()) == list(range(30))
    # with every sample a member, each row's maximum is its own (cosine) diagonal entry ~ 1
    assert fv[0] == pytest.approx(np.maximum(S.max(axis=1), 0).sum(), rel=1e-15)
    assert fv[0] == pytest.approx(30.0, rel=1e-2)


# ----------------------------------------------------------------------------- per-step exhaustive confirmation

def check_every_pick_by_enumeration(S, q, oj, ov):
    W, M = len(q), S.shape[0]
    A = [set() for _ in range(W)]
    J = set(range(W))
    R = set(range(M))
    t = 0
    while R and J:
        fJ = {j: brute_f(S, A[j]) for j in J}
        jstar = min(J, key=lambda j: (fJ[j], j))
        if len(A[jstar]) + 1 <= q[jstar]:
            vals = {v: brute_f(S, A[jstar] | {v}) for v in R}
            vstar = min(R, key=lambda v: (-vals[v], v))
            assert (oj[t], ov[t]) == (jstar, vstar), "step %d" % t
            A[jstar].add(vstar)
            R.remove(vstar)
            t += 1
        else:
            J.remove(jstar)
    assert t == len(oj)
    return A


@pytest.mark.parametrize("seed", range(6))
def test_every_pick_is_the_enumerated_argmin_argmax(seed):
    rng = np.random.default_rng(100 + seed)
    M = int(rng.integers(5, 12))
    W = int(rng.integers(1, 5))
    S = rand_sym_int(rng, M)
    q = orc.quotas(M, rng.uniform(0.5, 4.0, size=W))
    for variant in ("plain", "incremental"):
        assign, oj, ov, fv = orc.partition_class(S, q, variant)
        A = check_every_pick_by_enumeration(S, q.tolist(), oj.tolist(), ov.tolist())
        for j in range(W):
            assert fv[j] == brute_f(S, A[j])
            assert sorted(np.nonzero(assign == j)[0].tolist()) == sorted(A[j])


# ----------------------------------------------------------------------------- plain == incremental

@pytest.mark.parametrize("seed", range(5))
def test_incremental_equals_plain_int(seed):
    rng = np.random.default_rng(200 + seed)
    M, W = int(rng.integers(20, 70)), int(rng.integers(2, 7))
    S = rand_sym_int(rng, M, -300, 900)
    q = orc.quotas(M, rng.uniform(1, 8, size=W))
    a = orc.partition_class(S, q, "plain")
    b = orc.partition_class(S, q, "incremental")
    for x, y in zip(a, b):
        assert np.array_equal(x, y)


@pytest.mark.parametrize("seed", range(4))
def test_incremental_equals_plain_float(seed):
    from paper_2211_00839_b200.workloads import make_workload
    wl = make_workload("C4", L=1, M=48, d=64, seed=300 + seed)
    S = orc.similarity(wl.features)
    q = orc.quotas(48, wl.capacities[:5])
    a = orc.partition_class(S, q, "plain")
    b = orc.partition_class(S, q, "incremental")
    assert np.array_equal(a[0], b[0]) and np.array_equal(a[1], b[1]) and np.array_equal(a[2], b[2])
    assert np.array_equal(a[3], b[3])      # f is the same ascending sum of the same maxima in both


# ----------------------------------------------------------------------------- invariants of the output

@pytest.mark.parametrize("name,M,d", [("C1", 60, 32), ("C3", 50, 64)])
def test_partition_invariants(name, M, d):
    from paper_2211_00839_b200.workloads import make_workload
    wl = make_workload(name, L=3, M=M, d=d)
    res = orc.partition(wl.features, wl.labels, wl.capacities, wl.L, variant="incremental")
    # disjoint cover of every class (Section 3.1: A_i ^ A_j = 0, union = V_l)
    assert np.all(res.assignment >= 0) and np.all(res.assignment < wl.W)
    assert sorted(res.order.tolist()) == list(range(wl.N))
    for l in range(wl.L):
        ids = np.nonzero(wl.labels == l)[0]
        sizes = np.bincount(res.assignment[ids], minlength=wl.W)
        assert np.array_equal(sizes, res.quotas[l])            # |A_j^l| = C_{l,j}
        assert np.array_equal(res.quotas[l], res.quotas[0])    # same constraint for every (equal-sized) class
        o = res.class_offsets
        assert set(res.order[o[l]:o[l + 1]].tolist()) == set(ids.tolist())
    # tracked f equals f recomputed from the final assignment by the plain definition
    again = orc.objective(wl.features, wl.labels, res.assignment, wl.W, wl.L)
    if wl.dtype == "int8":
        assert np.array_equal(again, res.part_values)
    else:
        assert np.allclose(again, res.part_values, rtol=1e-12)


def test_gains_of_a_fixed_candidate_never_increase():
    rng = np.random.default_rng(7)
    S = rand_sym_int(rng, 14)
    q = [7, 7]
    assign, oj, ov, fv = orc.partition_class(S, q, "plain")
    members = [[], []]
    prev = [orc.gains_plain(S, []), orc.gains_plain(S, [])]
    for j, v in zip(oj, ov):
        members[j].append(int(v))
        g = orc.gains_plain(S, members[j])
        assert np.all(g <= prev[j])
        prev[j] = g


# ----------------------------------------------------------------------------- greedy bound against the brute-force optimum

@pytest.mark.parametrize("seed", range(4))
def test_cardinality_greedy_bound(seed):
    # one block with quota k: Algorithm 1 is then the classic greedy for max f(A), |A| <= k, whose
    # value is at least (1 - 1/e) of the optimum for a monotone submodular f.
    rng = np.random.default_rng(400 + seed)
    M, k = 11, 4
    S = rand_sym_int(rng, M, -10, 50)
    assign, oj, ov, fv = orc.partition_class(S, [k], "plain")
    assert len(ov) == k and np.count_nonzero(assign == 0) == k and np.count_nonzero(assign == -1) == M - k
    opt = max(brute_f(S, set(A)) for A in itertools.combinations(range(M), k))
    assert fv[0] >= (1.0 - 1.0 / math.e) * opt
    assert fv[0] <= opt


def test_min_block_value_vs_bruteforce_maxmin_recorded():
    # The paper states no bound for the partition itself; record greedy min_j f(A_j) against the best
    # quota-respecting partition found by enumeration (never better than the optimum, and positive).
    rng = np.random.default_rng(9)
    M, q = 8, [2, 3, 3]
    S = rand_sym_int(rng, M, 0, 40)
    assign, oj, ov, fv = orc.partition_class(S, q, "plain")
    best = -1
    for labels in itertools.product(range(3), repeat=M):
        if [labels.count(j) for j in range(3)] != q:
            continue
        val = min(brute_f(S, {v for v in range(M) if labels[v] == j}) for j in range(3))
        best = max(best, val)
    assert 0 < fv.min() <= best


# ----------------------------------------------------------------------------- replay checker

def test_replay_accepts_own_trace_and_flags_planted_mistakes():
    rng = np.random.default_rng(10)
    S = rand_sym_int(rng, 25, -50, 400)
    q = orc.quotas(25, [1, 2, 2])
    assign, oj, ov, fv = orc.partition_class(S, q, "plain")
    bad, stats, fv2 = orc.replay_class(S, q, oj, ov, 0.0)
    assert bad == -1 and stats.tolist() == [0, 0, 0, 0] and np.array_equal(fv, fv2)
    # swap two picks of different samples inside the trace: some step stops being the argmax
    ov2 = ov.copy()
    ov2[3], ov2[9] = ov2[9], ov2[3]
    bad, stats, _ = orc.replay_class(S, q, oj, ov2, 0.0)
    assert bad >= 0 and stats[1] > 0
    # reuse a sample: structural failure
    ov3 = ov.copy()
    ov3[5] = ov3[2]
    bad, _, _ = orc.replay_class(S, q, oj, ov3, 0.0)
    assert bad == -(5 + 2)
    # wrong block: not the argmin
    oj4 = oj.copy()
    t = 4
    oj4[t] = (oj4[t] + 1) % 3
    bad, stats, _ = orc.replay_class(S, q, oj4, ov, 0.0)
    assert bad != -1


def _replay_cases():
    return json.load(open(os.path.join(GOLDEN, "hand_traces.json")))["replay_cases"]


def _check_replay_case(S, q, oj, ov, objective, stats_want, first_failure, fvals):
    for tol_text, want_bad in first_failure.items():
        bad, stats, fv = orc.replay_class(S, q, oj, ov, float(tol_text), objective=objective)
        assert bad == want_bad, (tol_text, bad)
        # the deviations themselves do not depend on the tolerance, and they are the hand values, not just "small"
        assert stats[0] == stats_want["block_mismatches"] and stats[1] == stats_want["sample_mismatches"]
        assert stats[2] == stats_want["block_excess"][0] / stats_want["block_excess"][1]
        assert stats[3] == stats_want["gain_deficit"][0] / stats_want["gain_deficit"][1]
        assert fv.tolist() == fvals


@pytest.mark.parametrize("as_float", [False, True])
@pytest.mark.parametrize("case", _replay_cases(), ids=lambda c: c["name"])
def test_replay_tolerance_hand_worked(case, as_float):
    """The size of the teacher-forced checker's relative deviations, on pick sequences that deviate from
    the greedy one by amounts computed by hand (GreedyStep's argmax, Algorithm 1's argmin over blocks):
    a 5e-4 deficit passes at 1e-3 and fails at 1e-4 at the step that has it, and the reported worst
    deviations equal the hand values.  A mis-scaled, swapped or wrongly normalised `rel` fails here."""
    S = np.array(case["S"], dtype=np.float64 if as_float else np.int64)
    fv = [float(x) for x in case["fvals"]] if as_float else case["fvals"]
    _check_replay_case(S, case["quotas"], case["order_j"], case["order_v"], case["objective"], case["stats"],
                       case["first_failure"], fv)
    if "variant_b" in case:
        b = case["variant_b"]
        fvb = [float(x) for x in b["fvals_after"]] if as_float else b["fvals_after"]
        _check_replay_case(S, case["quotas"], b["order_j"], b["order_v"], case["objective"], b["stats"],
                           b["first_failure"], fvb)


@pytest.mark.parametrize("objective", ["facility", "cut"])
@pytest.mark.parametrize("seed", range(3))
def test_replay_rejects_planted_mistakes(objective, seed):
    """Both checkers against false acceptance: starting from the oracle's own trace of a random class,
    every planted mistake is reported, at the step it was planted or (for a swap) no later than it."""
    rng = np.random.default_rng(700 + seed)
    M = 24
    S = rand_sym_int(rng, M, -50, 400)
    if objective == "cut":
        np.fill_diagonal(S, 0)
    q = orc.quotas(M, [1, 2, 2, 1])
    assign, oj, ov, fv = orc.partition_class(S, q, "plain", objective=objective)
    bad, stats, fv2 = orc.replay_class(S, q, oj, ov, 0.0, objective=objective)
    assert bad == -1 and stats.tolist() == [0, 0, 0, 0] and np.array_equal(fv, fv2)
    # exchange two picked samples (different gains): the earlier step is no longer the argmax
    a, b = 3, 11
    ov2 = ov.copy()
    ov2[a], ov2[b] = ov2[b], ov2[a]
    bad, stats, _ = orc.replay_class(S, q, oj, ov2, 0.0, objective=objective)
    assert 0 <= bad <= a and stats[1] > 0 and stats[3] > 0
    assert orc.replay_class(S, q, oj, ov2, 1e9, objective=objective)[0] == -1     # only the tolerance lets it through
    # a sample picked twice: structural, whatever the tolerance
    ov3 = ov.copy()
    ov3[7] = ov3[2]
    assert orc.replay_class(S, q, oj, ov3, 1e9, objective=objective)[0] == -(7 + 2)
    # a block other than the argmin at a step where the values differ
    t = next(k for k in range(4, M) if len(set(oj[:k].tolist())) == 4)
    oj4 = oj.copy()
    oj4[t] = (oj4[t] + 1) % 4
    bad, stats, _ = orc.replay_class(S, q, oj4, ov, 0.0, objective=objective)
    assert bad in (t, -(t + 2)), (bad, t)         # not the argmin (values differ), or already full
    # a block beyond its quota: structural
    full = int(np.argmin(q))
    t_full = int(np.nonzero(oj == full)[0][-1])
    later = next(k for k in range(t_full + 1, M))
    oj5 = oj.copy()
    oj5[later] = full
    assert orc.replay_class(S, q, oj5, ov, 1e9, objective=objective)[0] == -(later + 2)
    # an index out of range
    ov6 = ov.copy()
    ov6[5] = M
    assert orc.replay_class(S, q, oj, ov6, 1e9, objective=objective)[0] == -(5 + 2)


# ----------------------------------------------------------------------------- Gaussian-kernel similarity (Section 4 item 2)

def test_gaussian_two_points_closed_form():
    # two points at distance delta: sigma = (0 + delta + delta + 0) / 4 = delta / 2, so the off-diagonal
    # similarity is exp(-delta^2 / (2 delta^2 / 4)) = exp(-2) whatever delta is
    for delta in (1, 7, 100):
        X = np.array([[0, 0, 0], [delta, 0, 0]], dtype=np.int8)
        S, sigma = orc.similarity_gaussian(X)
        assert sigma == pytest.approx(delta / 2.0, rel=1e-15)
        assert S[0, 0] == 1.0 and S[1, 1] == 1.0
        assert S[0, 1] == pytest.approx(math.exp(-2.0), rel=1e-14) and S[1, 0] == S[0, 1]


def test_gaussian_equidistant_points_closed_form():
    # M scaled one-hot vectors are pairwise at distance c*sqrt(2): sigma = delta (M-1)/M and every
    # off-diagonal similarity is exp(-M^2 / (2 (M-1)^2))
    M, c = 6, 9
    X = (c * np.eye(M, 8)).astype(np.int8)
    S, sigma = orc.similarity_gaussian(X)
    delta = c * math.sqrt(2.0)
    assert sigma == pytest.approx(delta * (M - 1) / M, rel=1e-14)
    off = math.exp(-M * M / (2.0 * (M - 1) ** 2))
    assert np.allclose(S[~np.eye(M, dtype=bool)], off, rtol=1e-13)
    assert np.array_equal(np.diag(S), np.ones(M))


def test_gaussian_matches_library_distances_and_is_scale_invariant():
    from scipy.spatial.distance import cdist
    from paper_2211_00839_b200.workloads import fp32_to_bf16_bits, bf16_bits_to_fp32
    rng = np.random.default_rng(12)
    X = rng.integers(-40, 41, size=(23, 17)).astype(np.int8)
    S, sigma = orc.similarity_gaussian(X)
    D = cdist(X.astype(np.float64), X.astype(np.float64))            # library routine for the distances
    assert sigma == pytest.approx(D.sum() / 23 ** 2, rel=1e-13)
    assert np.allclose(S, np.exp(-D ** 2 / (2 * sigma ** 2)), rtol=1e-12)
    assert np.array_equal(S, S.T) and np.all(S > 0) and np.all(S <= 1)
    # a larger distance never gives a larger similarity
    order = np.argsort(D[0])
    assert np.all(np.diff(S[0][order]) <= 1e-15)
    # doubling every feature doubles every distance and sigma: the similarities do not move
    S2, sigma2 = orc.similarity_gaussian((2 * X).astype(np.int8))
    assert sigma2 == pytest.approx(2 * sigma, rel=1e-14) and np.allclose(S2, S, rtol=1e-13)
    # translation does not matter either; and the bf16 variant sees the rounded values
    S3, _ = orc.similarity_gaussian((X + 5).astype(np.int8))
    assert np.allclose(S3, S, rtol=1e-13)
    x = rng.standard_normal((9, 12)).astype(np.float32)
    bits = fp32_to_bf16_bits(x)
    Sb, sb = orc.similarity_gaussian(bits)
    Db = cdist(bf16_bits_to_fp32(bits).astype(np.float64), bf16_bits_to_fp32(bits).astype(np.float64))
    assert sb == pytest.approx(Db.sum() / 81, rel=1e-13)
    assert np.allclose(Sb, np.exp(-Db ** 2 / (2 * sb ** 2)), rtol=1e-12)


def test_gaussian_coincident_points():
    X = np.full((4, 5), 3, dtype=np.int8)
    S, sigma = orc.similarity_gaussian(X)
    assert sigma == 0.0 and np.array_equal(S, np.ones((4, 4)))


def test_partition_with_gaussian_similarity_keeps_the_invariants():
    from paper_2211_00839_b200.workloads import make_workload
    wl = make_workload("C1", L=2, M=40, d=16)
    res = orc.partition(wl.features, wl.labels, wl.capacities, wl.L, variant="plain", similarity_kind="gaussian")
    inc = orc.partition(wl.features, wl.labels, wl.capacities, wl.L, variant="incremental", similarity_kind="gaussian")
    assert np.array_equal(res.assignment, inc.assignment) and np.array_equal(res.order, inc.order)
    assert res.part_values.dtype == np.float64
    for l in range(wl.L):
        ids = np.nonzero(wl.labels == l)[0]
        assert np.array_equal(np.bincount(res.assignment[ids], minlength=wl.W), res.quotas[l])
    again = orc.objective(wl.features, wl.labels, res.assignment, wl.W, wl.L, similarity_kind="gaussian")
    assert np.allclose(again, res.part_values, rtol=1e-12)
    # with S in (0, 1] and S[i][i] = 1, a block that holds everything covers every point fully
    S, _ = orc.similarity_gaussian(wl.features[wl.labels == 0])
    assert orc.f_plain(S, list(range(S.shape[0]))) == pytest.approx(S.shape[0], rel=1e-15)


# ----------------------------------------------------------------------------- graph-cut objective (Section 4 item 2)

def brute_cut(S, A):
    A = sorted(A)
    out = [v for v in range(S.shape[0]) if v not in A]
    if not A or not out:
        return S.dtype.type(0)
    return S[np.ix_(out, A)].sum()


def test_graph_cut_closed_forms():
    M = 7
    S = np.ones((M, M), dtype=np.int64)
    for n in range(M + 1):
        assert orc.f_plain(S, list(range(n)), "cut") == (M - n) * n          # |V \ A| * |A| unit edges
    assert orc.f_plain((5 * np.eye(M)).astype(np.int64), [1, 3], "cut") == 0   # no edges between distinct samples
    # rows are the outside samples, columns the members: a non-symmetric S exposes a transposed operand
    S = np.array([[0, 1], [5, 0]], dtype=np.int64)
    assert orc.f_plain(S, [0], "cut") == 5 and orc.f_plain(S, [1], "cut") == 1
    # not monotone: the full set cuts nothing
    rng = np.random.default_rng(21)
    S = rand_sym_int(rng, 9, 0, 30)
    assert orc.f_plain(S, list(range(9)), "cut") == 0 and orc.f_plain(S, [], "cut") == 0
    for A in ([2], [0, 5, 7], [1, 2, 3, 4, 8]):
        assert orc.f_plain(S, A, "cut") == brute_cut(S, A)
        g = orc.gains_plain(S, A, "cut")
        for v in range(9):
            if v not in A:
                assert g[v] == brute_cut(S, A + [v]) - brute_cut(S, A)


@pytest.mark.parametrize("seed", range(5))
def test_graph_cut_every_pick_enumerated_and_variants_agree(seed):
    rng = np.random.default_rng(500 + seed)
    M = int(rng.integers(5, 12))
    W = int(rng.integers(1, 4))
    S = rand_sym_int(rng, M, -10, 40)
    q = orc.quotas(M, rng.uniform(0.5, 3.0, size=W)).tolist()
    plain = orc.partition_class(S, q, "plain", objective="cut")
    inc = orc.partition_class(S, q, "incremental", objective="cut")
    for x, y in zip(plain, inc):
        assert np.array_equal(x, y)
    assign, oj, ov, fv = plain
    A = [set() for _ in range(W)]
    J, R, t = set(range(W)), set(range(M)), 0
    while R and J:
        fJ = {j: brute_cut(S, A[j]) for j in J}
        jstar = min(J, key=lambda j: (fJ[j], j))
        if len(A[jstar]) + 1 <= q[jstar]:
            vals = {v: brute_cut(S, A[jstar] | {v}) for v in R}
            vstar = min(R, key=lambda v: (-vals[v], v))
            assert (oj[t], ov[t]) == (jstar, vstar)
            A[jstar].add(vstar); R.remove(vstar); t += 1
        else:
            J.remove(jstar)
    assert t == len(oj)
    for j in range(W):
        assert fv[j] == brute_cut(S, A[j])
    bad, stats, fv2 = orc.replay_class(S, q, oj, ov, 0.0, objective="cut")
    assert bad == -1 and stats.tolist() == [0, 0, 0, 0] and np.array_equal(fv2, fv)


def test_graph_cut_incremental_close_to_plain_in_double_and_invariants():
    from paper_2211_00839_b200.workloads import make_workload
    wl = make_workload("C4", L=2, M=40, d=32, seed=77)
    res = orc.partition(wl.features, wl.labels, wl.capacities[:4], wl.L, variant="plain", objective="cut")
    inc = orc.partition(wl.features, wl.labels, wl.capacities[:4], wl.L, variant="incremental", objective="cut")
    assert np.array_equal(res.assignment, inc.assignment) and np.array_equal(res.order, inc.order)
    assert np.allclose(res.part_values, inc.part_values, rtol=1e-12)
    for l in range(wl.L):
        ids = np.nonzero(wl.labels == l)[0]
        assert np.array_equal(np.bincount(res.assignment[ids], minlength=4), res.quotas[l])
    again = orc.objective(wl.features, wl.labels, res.assignment, 4, wl.L, objective="cut")
    assert np.allclose(again, res.part_values, rtol=1e-12)


# ----------------------------------------------------------------------------- downstream hook: worker lists, batch sizes

def test_worker_lists_hand_example():
    """Seven samples, three workers, written out by hand."""
    a = np.array([2, 0, 1, 0, 2, 2, 1], dtype=np.int32)
    off, idx = orc.worker_lists(a, 3)
    assert off.tolist() == [0, 2, 4, 7]
    assert idx.tolist() == [1, 3, 2, 6, 0, 4, 5]
    off, idx = orc.worker_lists(a, 4)                      # a worker that got nothing
    assert off.tolist() == [0, 2, 4, 7, 7]


def test_worker_lists_are_a_stable_partition_with_quota_sizes():
    """On a real partition: the lists are disjoint, cover the dataset, are ascending, agree with a stable
    argsort (library routine), and worker j holds sum_l C_{l,j} samples (Algorithm 1's constraint)."""
    from paper_2211_00839_b200.workloads import make_workload
    wl = make_workload("C1")
    ref = orc.partition(wl.features, wl.labels, wl.capacities, wl.L, variant="incremental")
    off, idx = orc.worker_lists(ref.assignment, wl.W)
    assert sorted(idx.tolist()) == list(range(wl.N))
    assert np.array_equal(idx, np.argsort(ref.assignment, kind="stable"))
    for j in range(wl.W):
        mine = idx[off[j]:off[j + 1]]
        assert np.all(np.diff(mine) > 0) and np.all(ref.assignment[mine] == j)
        assert len(mine) == int(ref.quotas[:, j].sum())
    assert (off[1:] - off[:-1]).tolist() == [50, 50, 100, 200]   # 2 classes x (25, 25, 50, 100)


def test_batch_sizes_closed_forms():
    assert orc.batch_sizes(32, [1, 1, 2, 4]).tolist() == [32, 32, 64, 128]
    # the ratio as Algorithm 2 prints it: B r_1 / r_i
    assert orc.batch_sizes(32, [1, 1, 2, 4], rule="printed").tolist() == [32, 32, 16, 8]
    assert orc.batch_sizes(10, [4, 1, 3], rule="printed").tolist() == [10, 40, 13]      # 13.33 -> 13
    assert orc.batch_sizes(1, [1, 8], rule="printed").tolist() == [1, 1]
    assert orc.batch_sizes(32, [2, 1, 4]).tolist() == [32, 16, 64]          # relative to worker 1
    assert orc.batch_sizes(10, [4, 1, 3]).tolist() == [10, 3, 8]            # 2.5 -> 3, 7.5 -> 8: halves round up
    assert orc.batch_sizes(1, [8, 1]).tolist() == [1, 1]                    # never below one sample
    b = orc.batch_sizes(64, [1.0, 2.5, 3.5])
    assert b.tolist() == [64, 160, 224] and b[1] / b[0] == 2.5
