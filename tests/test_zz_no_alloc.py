"""The allocation-free objective entry point against the workspace-based one.

rcd_objective_class_static is for callers that cannot allocate device memory (a fixed memory
budget, or a region where the CUDA allocator must not be touched): its scratch is an array built
into the library.  Here both entry points get the same single-class input, twice in a row (the
second call reuses the array with the first call's leftovers in it), and must agree: exactly for
int8 features, and to the tolerance of the other objective tests for bf16 features.

This file sorts last on purpose, so a run that stops at the first failure has already run
everything else; it also passes when run alone in a fresh process.
"""
import numpy as np
import pytest

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("name,M,d,W", [("C2", 700, 128, 8), ("C4", 450, 96, 32), ("C5", 300, 128, 64)])
def test_static_scratch_objective_matches_workspace_objective_twice(name, M, d, W):
    import torch
    from paper_2211_00839_b200 import binding as rcd
    from paper_2211_00839_b200.workloads import make_workload
    from oracle import rcd_oracle as orc

    dev = torch.device("cuda", 0)
    with rcd.Context(0) as ctx:
        for call, seed in enumerate((21, 22)):            # two calls in a row, different data
            wl = make_workload(name, L=1, M=M, d=d, seed=seed, shuffle=False)
            rng = np.random.default_rng(seed)
            assignment = torch.from_numpy(rng.integers(-1, W, size=M).astype(np.int32)).to(dev)
            X = rcd.features_to_torch(wl.features, device=dev)
            y = torch.zeros(M, dtype=torch.int32, device=dev)
            want_vals, want_total = ctx.rcd_objective(X, y, assignment, W, 1)
            S = ctx.rcd_similarity(X)[0]
            vdt = torch.int64 if wl.dtype == "int8" else torch.float64
            vals = torch.full((W,), -7, dtype=vdt, device=dev)
            total = torch.full((1,), -7, dtype=vdt, device=dev)
            rcd.rcd_objective_class_static(ctx, S, assignment, W, vals, total)
            ctx.sync_status()
            # ... and the oracle's plain definition of f on the same class
            So = orc.similarity(wl.features)
            a_host = assignment.cpu().numpy()
            plain = np.array([orc.f_plain(So, np.nonzero(a_host == j)[0]) for j in range(W)])
            if wl.dtype == "int8":
                assert torch.equal(vals, want_vals[0]), "call %d" % call
                assert int(total[0]) == int(want_total[0])
                assert np.array_equal(vals.cpu().numpy(), plain)
            else:
                assert torch.allclose(vals, want_vals[0], rtol=1e-5, atol=1e-7), "call %d" % call
                assert float(total[0]) == pytest.approx(float(want_total[0]), rel=1e-5)
                assert np.allclose(vals.cpu().numpy(), plain, rtol=1e-5, atol=1e-7)


def test_static_scratch_at_its_size_limit():
    """ceil(M/64) * W * 8 exactly 1 MiB is served (and equals the plain definition); one row block more is refused."""
    import ctypes as C
    import torch
    from paper_2211_00839_b200 import binding as rcd
    from oracle import rcd_oracle as orc
    dev = torch.device("cuda", 0)
    W = 1024
    M = 64 * 128                                     # 128 row blocks * 1024 * 8 bytes = 1 MiB
    rng = np.random.default_rng(31)
    d = 16
    X = rng.integers(-20, 21, size=(M, d)).astype(np.int8)
    a_host = rng.integers(-1, W, size=M).astype(np.int32)
    with rcd.Context(0) as ctx:
        S = ctx.rcd_similarity(torch.from_numpy(X).to(dev))[0]
        a = torch.from_numpy(a_host).to(dev)
        vals = torch.full((W,), -7, dtype=torch.int64, device=dev)
        total = torch.full((1,), -7, dtype=torch.int64, device=dev)
        rcd.rcd_objective_class_static(ctx, S, a, W, vals, total)
        ctx.sync_status()
        So = orc.similarity(X)
        # plain definition, vectorised per block: sum over rows of the clamped maximum over the block's members
        want = np.zeros(W, dtype=np.int64)
        for j in range(W):
            mem = np.nonzero(a_host == j)[0]
            if len(mem):
                want[j] = np.maximum(So[:, mem].max(axis=1), 0).sum()
        for j in (0, 1, 511, 1023):
            assert want[j] == orc.f_plain(So, np.nonzero(a_host == j)[0])
        assert np.array_equal(vals.cpu().numpy(), want) and int(total[0]) == int(want.sum())
        Mbig = M + 1                                 # one more row block: 129 * 1024 * 8 > 1 MiB
        st = rcd.lib.rcd_objective_class_static(ctx._h, C.c_void_p(S.data_ptr()), rcd.RCD_FEAT_I8, Mbig, Mbig,
                                                C.c_void_p(a.data_ptr()), W, C.c_void_p(vals.data_ptr()),
                                                C.c_void_p(total.data_ptr()), None)
        assert st == 2


def test_static_scratch_refuses_a_graph_cut_context():
    import ctypes as C
    import torch
    from paper_2211_00839_b200 import binding as rcd
    dev = torch.device("cuda", 0)
    with rcd.Context(0, objective=rcd.RCD_OBJ_GRAPH_CUT) as ctx:
        S = torch.zeros((8, 8), dtype=torch.int32, device=dev)
        a = torch.zeros(8, dtype=torch.int32, device=dev)
        vals = torch.zeros(2, dtype=torch.int64, device=dev)
        total = torch.zeros(1, dtype=torch.int64, device=dev)
        st = rcd.lib.rcd_objective_class_static(ctx._h, C.c_void_p(S.data_ptr()), rcd.RCD_FEAT_I8, 8, 8,
                                                C.c_void_p(a.data_ptr()), 2, C.c_void_p(vals.data_ptr()),
                                                C.c_void_p(total.data_ptr()), None)
        assert st == 2 and b"facility" in rcd.lib.rcd_last_error(ctx._h)


def test_static_scratch_rejects_sizes_beyond_its_array():
    import torch
    from paper_2211_00839_b200 import binding as rcd
    dev = torch.device("cuda", 0)
    with rcd.Context(0) as ctx:
        M, W = 64 * 200, 1024                       # 200 row blocks * 1024 * 8 bytes > 1 MiB
        S = torch.zeros((8, 8), dtype=torch.int32, device=dev)          # never read: the call must refuse first
        a = torch.zeros(8, dtype=torch.int32, device=dev)
        vals = torch.zeros(W, dtype=torch.int64, device=dev)
        total = torch.zeros(1, dtype=torch.int64, device=dev)
        import ctypes as C
        st = rcd.lib.rcd_objective_class_static(ctx._h, C.c_void_p(S.data_ptr()), rcd.RCD_FEAT_I8, M, M,
                                                C.c_void_p(a.data_ptr()), W, C.c_void_p(vals.data_ptr()),
                                                C.c_void_p(total.data_ptr()), None)
        assert st == 2
        assert b"scratch" in rcd.lib.rcd_last_error(ctx._h)
