"""CPU-side checks of the C-ABI library: it loads, exports what include/rcd.h declares, and its
host-only logic (quotas) agrees with the oracle.  No compute call is made here."""
import ctypes
import os
import re

import numpy as np
import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def binding():
    from paper_2211_00839_b200 import build
    build.build()
    from paper_2211_00839_b200 import binding as b
    return b


def test_library_loads_and_exports_every_declared_symbol(binding):
    header = open(os.path.join(ROOT, "include", "rcd.h")).read()
    declared = sorted(set(re.findall(r"RCD_API[^;(]*?\b(rcd_[a-z_]+)\s*\(", header)))
    assert declared, "no declarations found in the header"
    assert sorted(binding.EXPORTS) == declared
    lib = ctypes.CDLL(binding.LIB_PATH)
    for name in declared:
        assert hasattr(lib, name), name
    assert "sm_100a" in binding.rcd_version()


def test_quotas_match_oracle_and_closed_forms(binding):
    from oracle import rcd_oracle as orc
    assert binding.rcd_quotas(200, [1, 1, 2, 4]).tolist() == [25, 25, 50, 100]
    assert binding.rcd_quotas(5000, [1, 1, 1, 1, 2, 2, 4, 4]).tolist() == [313, 313, 312, 312, 625, 625, 1250, 1250]
    caps = [2.0 ** (j // 16) for j in range(64)]
    assert binding.rcd_quotas(1300, caps).tolist() == [6] * 4 + [5] * 12 + [11] * 16 + [22] * 16 + [43] * 16
    rng = np.random.default_rng(11)
    for _ in range(300):
        W = int(rng.integers(1, 70))
        M = int(rng.integers(0, 6000))
        r = rng.uniform(0.05, 9.0, size=W)
        if rng.random() < 0.3:
            r = np.round(r * 2) / 2 + 0.5
        a = binding.rcd_quotas(M, r)
        assert a.sum() == M
        assert np.array_equal(a, orc.quotas(M, r))


def test_batch_sizes_match_oracle_and_closed_forms(binding):
    from oracle import rcd_oracle as orc
    assert binding.rcd_batch_sizes(32, [1, 1, 2, 4]).tolist() == [32, 32, 64, 128]
    assert binding.rcd_batch_sizes(10, [4, 1, 3]).tolist() == [10, 3, 8]
    assert binding.rcd_batch_sizes(32, [1, 1, 2, 4], rule=binding.RCD_BATCH_AS_PRINTED).tolist() == [32, 32, 16, 8]
    rng2 = np.random.default_rng(77)
    for _ in range(50):
        r2 = rng2.uniform(0.2, 9.0, size=int(rng2.integers(1, 20)))
        B2 = int(rng2.integers(1, 500))
        assert np.array_equal(binding.rcd_batch_sizes(B2, r2, rule=binding.RCD_BATCH_AS_PRINTED), orc.batch_sizes(B2, r2, rule="printed"))
    rng = np.random.default_rng(12)
    for _ in range(200):
        W = int(rng.integers(1, 70))
        B = int(rng.integers(1, 2000))
        r = np.round(rng.uniform(0.05, 9.0, size=W) * 4) / 4 + 0.25
        assert np.array_equal(binding.rcd_batch_sizes(B, r), orc.batch_sizes(B, r))
    for B, caps in ((0, [1.0]), (8, [1.0, 0.0]), (8, [float("nan"), 1.0])):
        with pytest.raises(binding.RcdError):
            binding.rcd_batch_sizes(B, caps)


def test_quotas_reject_bad_arguments(binding):
    for caps in ([1.0, 0.0], [1.0, -2.0], [float("nan")], [float("inf"), 1.0]):
        with pytest.raises(binding.RcdError):
            binding.rcd_quotas(10, caps)
    with pytest.raises(binding.RcdError):
        binding.rcd_quotas(-1, [1.0])


def test_context_needs_a_gpu(binding):
    import torch
    if torch.cuda.is_available():
        pytest.skip("a GPU is present")
    with pytest.raises(binding.RcdError):
        binding.Context(0)


def test_no_oracle_in_the_product_path():
    """The package and bench's own arm must not import the oracle."""
    pkg = os.path.join(ROOT, "paper_2211_00839_b200")
    for dirpath, _, files in os.walk(pkg):
        for f in files:
            if f.endswith((".py", ".cu", ".h", ".cuh")):
                text = open(os.path.join(dirpath, f)).read()
                assert "oracle" not in text.lower() or f == "workloads.py" and "oracle's tests" in text, f


def test_quotas_decimal_grid_agrees_with_oracle_and_never_overshoots(binding):
    """Capacities that are not representable in binary (tenths), every pair and a sample of triples, M up to 60: the
    library's apportionment (ranked by a stable sort) equals the oracle's (repeated selection), the quotas add up to
    M, and the integer parts of the shares never add up to more than M -- the branch that would take samples back is
    not reached by any of these inputs."""
    import itertools
    import math
    from oracle import rcd_oracle as orc
    vals = [k / 10 for k in range(1, 31)]
    cases = list(itertools.product(vals, repeat=2)) + list(itertools.product(vals[::3], repeat=3))
    for r in cases:
        total = 0.0
        for x in r:
            total = total + x
        for M in (1, 7, 10, 33, 60):
            assert sum(math.floor(M * x / total) for x in r) <= M
            q = binding.rcd_quotas(M, r)
            assert q.sum() == M and np.array_equal(q, orc.quotas(M, r))
