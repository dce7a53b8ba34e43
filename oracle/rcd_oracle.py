"""ctypes front end of the CPU oracle (TEST INFRASTRUCTURE, not part of the product).

The arithmetic lives in ``rcd_oracle.c`` / ``rcd_oracle_typed.inc`` (plain C,
single-threaded, int64 or double).  This file only compiles and loads that
code, splits a dataset into classes (Algorithm 1, "Split the ground set V into
L sets according to class labels"), calls the per-class routines, and joins the
per-class blocks into one assignment vector ("Joint subset", Algorithm 1).

Nothing in the CUDA library imports this module and this module imports
nothing from the library.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from concurrent.futures import ThreadPoolExecutor
from typing import List, Optional, Sequence, Tuple

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = [os.path.join(_HERE, "rcd_oracle.c"), os.path.join(_HERE, "rcd_oracle_typed.inc")]
_SO = os.path.join(_HERE, "librcd_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (no fast-math, no FP contraction)."""
    newest = max(os.path.getmtime(p) for p in _SRC)
    if force or not os.path.exists(_SO) or os.path.getmtime(_SO) < newest:
        tmp = _SO + ".tmp.%d" % os.getpid()
        subprocess.check_call(["gcc", "-O2", "-std=c99", "-fPIC", "-shared", "-fno-fast-math",
                               "-ffp-contract=off", "-o", tmp, _SRC[0], "-lm"])
        os.replace(tmp, _SO)
    return _SO


def _load():
    global _lib
    if _lib is not None:
        return _lib
    lib = C.CDLL(build())
    i64, i32, dbl = C.c_int64, C.c_int32, C.c_double
    P = C.c_void_p
    lib.rcd_oracle_similarity_i8.argtypes = [P, i64, i64, P]
    lib.rcd_oracle_similarity_bf16.argtypes = [P, i64, i64, P]
    lib.rcd_oracle_quotas.argtypes = [i64, P, i32, P]
    lib.rcd_oracle_gaussian_i8.argtypes = [P, i64, i64, P, P]
    lib.rcd_oracle_gaussian_bf16.argtypes = [P, i64, i64, P, P]
    for suf, ret in (("i64", i64), ("f64", dbl)):
        f = getattr(lib, "rcd_oracle_f_" + suf)
        f.argtypes = [P, i64, P, i64]
        f.restype = ret
        fc = getattr(lib, "rcd_oracle_f_cut_" + suf)
        fc.argtypes = [P, i64, P, i64]
        fc.restype = ret
        for name in ("rcd_oracle_partition_plain_", "rcd_oracle_partition_incremental_"):
            g = getattr(lib, name + suf)
            g.argtypes = [P, i64, i32, P, P, P, P, P, i64, C.c_int]
            g.restype = i64
        for name in ("rcd_oracle_replay_", "rcd_oracle_replay_cut_"):
            r = getattr(lib, name + suf)
            r.argtypes = [P, i64, i32, P, P, P, i64, dbl, P, P]
            r.restype = i64
        q = getattr(lib, "rcd_oracle_gains_" + suf)
        q.argtypes = [P, i64, P, i64, P, C.c_int]
        q.restype = None
    _lib = lib
    return lib


def _ptr(a: np.ndarray):
    return a.ctypes.data_as(C.c_void_p)


def _suffix(S: np.ndarray) -> str:
    if S.dtype == np.int64:
        return "i64"
    if S.dtype == np.float64:
        return "f64"
    raise TypeError("S must be int64 or float64, got %s" % S.dtype)


# --------------------------------------------------------------------------- per-class pieces

def similarity(X: np.ndarray) -> np.ndarray:
    """S = X X^T for one class.  int8 -> int64 (exact); uint16 bf16 bits -> float64."""
    lib = _load()
    X = np.ascontiguousarray(X)
    M, d = X.shape
    if X.dtype == np.int8:
        S = np.empty((M, M), dtype=np.int64)
        lib.rcd_oracle_similarity_i8(_ptr(X), M, d, _ptr(S))
    elif X.dtype == np.uint16:
        S = np.empty((M, M), dtype=np.float64)
        lib.rcd_oracle_similarity_bf16(_ptr(X), M, d, _ptr(S))
    else:
        raise TypeError("features must be int8 or uint16 (bf16 bits)")
    return S


def similarity_gaussian(X: np.ndarray):
    """Gaussian-kernel similarity of one class and its bandwidth: (S float64 [M, M], sigma)."""
    lib = _load()
    X = np.ascontiguousarray(X)
    M, d = X.shape
    S = np.empty((M, M), dtype=np.float64)
    sigma = C.c_double(0.0)
    if X.dtype == np.int8:
        lib.rcd_oracle_gaussian_i8(_ptr(X), M, d, _ptr(S), C.byref(sigma))
    elif X.dtype == np.uint16:
        lib.rcd_oracle_gaussian_bf16(_ptr(X), M, d, _ptr(S), C.byref(sigma))
    else:
        raise TypeError("features must be int8 or uint16 (bf16 bits)")
    return S, float(sigma.value)


def class_similarity(X: np.ndarray, kind: str = "dot") -> np.ndarray:
    """S of one class for the chosen similarity ("dot": dot product / cosine; "gaussian")."""
    if kind == "dot":
        return similarity(X)
    if kind == "gaussian":
        return similarity_gaussian(X)[0]
    raise ValueError(kind)


def quotas(M: int, capacities: Sequence[float]) -> np.ndarray:
    """Integer quotas C_{l,j} of one class of M samples (largest-remainder rule)."""
    lib = _load()
    r = np.ascontiguousarray(capacities, dtype=np.float64)
    out = np.empty(len(r), dtype=np.int32)
    lib.rcd_oracle_quotas(int(M), _ptr(r), len(r), _ptr(out))
    return out


OBJECTIVES = {"facility": 0, "cut": 1}


def f_plain(S: np.ndarray, members: Sequence[int], objective: str = "facility"):
    """f(A) from the plain definition: facility location, or graph cut (Section 4 item 2)."""
    lib = _load()
    S = np.ascontiguousarray(S)
    m = np.ascontiguousarray(members, dtype=np.int32)
    name = "rcd_oracle_f_cut_" if OBJECTIVES[objective] == 1 else "rcd_oracle_f_"
    return getattr(lib, name + _suffix(S))(_ptr(S), S.shape[0], _ptr(m), len(m))


def gains_plain(S: np.ndarray, members: Sequence[int], objective: str = "facility") -> np.ndarray:
    """f(A u {v}) - f(A) for every v, from the plain definition."""
    lib = _load()
    S = np.ascontiguousarray(S)
    m = np.ascontiguousarray(members, dtype=np.int32)
    out = np.empty(S.shape[0], dtype=S.dtype)
    getattr(lib, "rcd_oracle_gains_" + _suffix(S))(_ptr(S), S.shape[0], _ptr(m), len(m), _ptr(out), OBJECTIVES[objective])
    return out


def partition_class(S: np.ndarray, C_quota: Sequence[int], variant: str = "plain", max_picks: int = -1,
                    objective: str = "facility"):
    """Algorithm 1 on one class.  Returns (assign[M], order_j[T], order_v[T], fvals[W]).

    ``max_picks >= 0`` stops the loop after that many picks (bounded timing sample)."""
    lib = _load()
    S = np.ascontiguousarray(S)
    M = S.shape[0]
    q = np.ascontiguousarray(C_quota, dtype=np.int32)
    W = len(q)
    assign = np.empty(M, dtype=np.int32)
    oj = np.empty(max(M, 1), dtype=np.int32)
    ov = np.empty(max(M, 1), dtype=np.int32)
    fv = np.empty(W, dtype=S.dtype)
    name = {"plain": "rcd_oracle_partition_plain_", "incremental": "rcd_oracle_partition_incremental_"}[variant]
    T = getattr(lib, name + _suffix(S))(_ptr(S), M, W, _ptr(q), _ptr(assign), _ptr(oj), _ptr(ov), _ptr(fv),
                                         int(max_picks), OBJECTIVES[objective])
    return assign, oj[:T].copy(), ov[:T].copy(), fv


def replay_class(S: np.ndarray, C_quota: Sequence[int], order_j: Sequence[int], order_v: Sequence[int],
                 rel_tol: float, objective: str = "facility"):
    """Teacher-forced check of a pick sequence.  Returns (first_bad_step or -1, stats[4], fvals[W])."""
    lib = _load()
    S = np.ascontiguousarray(S)
    q = np.ascontiguousarray(C_quota, dtype=np.int32)
    oj = np.ascontiguousarray(order_j, dtype=np.int32)
    ov = np.ascontiguousarray(order_v, dtype=np.int32)
    stats = np.zeros(4, dtype=np.float64)
    fv = np.empty(len(q), dtype=S.dtype)
    rname = "rcd_oracle_replay_cut_" if OBJECTIVES[objective] == 1 else "rcd_oracle_replay_"
    bad = getattr(lib, rname + _suffix(S))(_ptr(S), S.shape[0], len(q), _ptr(q), _ptr(oj), _ptr(ov),
                                                         len(oj), float(rel_tol), _ptr(stats), _ptr(fv))
    return int(bad), stats, fv


# --------------------------------------------------------------------------- whole dataset

def split_by_label(labels: np.ndarray, L: int) -> List[np.ndarray]:
    """V -> V_1..V_L; inside a class the samples keep their dataset order."""
    groups: List[List[int]] = [[] for _ in range(L)]
    for idx, lab in enumerate(np.asarray(labels).tolist()):
        groups[lab].append(idx)
    return [np.asarray(g, dtype=np.int64) for g in groups]


class PartitionResult:
    def __init__(self, N: int, L: int, W: int, value_dtype):
        self.assignment = np.full(N, -1, dtype=np.int32)       # block of every sample
        self.order = np.full(N, -1, dtype=np.int32)            # per class (class-major), global ids in pick order
        self.order_block = np.full(N, -1, dtype=np.int32)      # block of each pick, same layout
        self.class_offsets = np.zeros(L + 1, dtype=np.int64)
        self.part_values = np.zeros((L, W), dtype=value_dtype)  # f(A_j^l)
        self.quotas = np.zeros((L, W), dtype=np.int32)

    @property
    def total(self):
        return self.part_values.sum()


def partition(features: np.ndarray, labels: np.ndarray, capacities: Sequence[float], L: int,
              variant: str = "incremental", threads: int = 1,
              classes: Optional[Sequence[int]] = None, max_picks: int = -1,
              similarity_kind: str = "dot", objective: str = "facility") -> PartitionResult:
    """Algorithm 1 over the whole dataset: classes handled one after another
    (or one per thread: they are independent), blocks joined at the end.

    ``classes`` restricts the run to some classes (others stay -1 / zero);
    ``max_picks`` truncates every class's loop (bounded timing sample)."""
    features = np.ascontiguousarray(features)
    N = features.shape[0]
    W = len(capacities)
    vdt = np.int64 if (features.dtype == np.int8 and similarity_kind == "dot") else np.float64
    groups = split_by_label(labels, L)
    res = PartitionResult(N, L, W, vdt)
    res.class_offsets[1:] = np.cumsum([len(g) for g in groups])
    todo = list(range(L)) if classes is None else list(classes)

    def one(l: int):
        ids = groups[l]
        M = len(ids)
        q = quotas(M, capacities)
        if M == 0:
            return l, q, None
        S = class_similarity(features[ids], similarity_kind)
        return l, q, partition_class(S, q, variant, max_picks, objective)

    if threads > 1:
        with ThreadPoolExecutor(max_workers=threads) as ex:
            outs = list(ex.map(one, todo))
    else:
        outs = [one(l) for l in todo]
    for l, q, out in outs:
        res.quotas[l] = q
        if out is None:
            continue
        assign, oj, ov, fv = out
        ids = groups[l]
        res.assignment[ids] = assign
        o = int(res.class_offsets[l])
        res.order[o:o + len(ov)] = ids[ov]
        res.order_block[o:o + len(oj)] = oj
        res.part_values[l] = fv
    return res


def objective(features: np.ndarray, labels: np.ndarray, assignment: np.ndarray, W: int, L: int,
              similarity_kind: str = "dot", objective: str = "facility") -> np.ndarray:
    """f(A_j^l) for all (l, j), recomputed from the plain definition given an assignment."""
    features = np.ascontiguousarray(features)
    vdt = np.int64 if (features.dtype == np.int8 and similarity_kind == "dot") else np.float64
    out = np.zeros((L, W), dtype=vdt)
    groups = split_by_label(labels, L)
    for l, ids in enumerate(groups):
        if len(ids) == 0:
            continue
        S = class_similarity(features[ids], similarity_kind)
        a = np.asarray(assignment)[ids]
        for j in range(W):
            out[l, j] = f_plain(S, np.nonzero(a == j)[0], objective)
    return out


# ----------------------------------------------------------------------------- downstream hook (Algorithm 2, initialisation)

def worker_lists(assignment: np.ndarray, W: int) -> Tuple[np.ndarray, np.ndarray]:
    """The local subset of every worker (Algorithm 2: worker i "imports the local subset xi_i from the
    subsets A_1 .. A_N"): worker j's list is every dataset index whose block is j, in ascending order.
    Returns (offsets [W+1], indices [N]) with worker j's list at indices[offsets[j]:offsets[j+1]].
    Plain definition, one pass per worker."""
    assignment = np.asarray(assignment)
    lists = []
    for j in range(W):
        mine = [i for i in range(len(assignment)) if assignment[i] == j]
        lists.append(np.asarray(mine, dtype=np.int32))
    offsets = np.zeros(W + 1, dtype=np.int64)
    for j in range(W):
        offsets[j + 1] = offsets[j] + len(lists[j])
    indices = np.concatenate(lists) if lists else np.zeros(0, np.int32)
    return offsets, indices.astype(np.int32)


def batch_sizes(B: int, capacities: Sequence[float], rule: str = "proportional") -> np.ndarray:
    """Per-worker batch sizes of Algorithm 2's initialisation.  The text below Algorithm 2 makes the batch
    size of a worker proportional to its processing speed (rule "proportional": b_i = B * r_i / r_1 with worker 1
    the reference); the algorithm's own line prints the inverse ratio (rule "printed": b_i = B * r_1 / r_i).
    Rounded half up to an integer, at least 1."""
    r = [float(x) for x in capacities]
    out = []
    for ri in r:
        x = float(B) * ri / r[0] if rule == "proportional" else float(B) * r[0] / ri
        out.append(max(1, int(np.floor(x + 0.5))))
    return np.asarray(out, dtype=np.int64)
