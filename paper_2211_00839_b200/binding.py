"""ctypes binding of the C-ABI library declared in ``include/rcd.h``.

Argument marshalling only: every step of the computation runs in the CUDA
kernels of ``librcd.so``.  PyTorch supplies device memory and streams.  If the
compiled library is missing, importing this module raises; there is no CPU
fallback of any kind.

The functions keep the names of the C entry points (``rcd_similarity``,
``rcd_partition``, ``rcd_partition_host``, ``rcd_objective``, ``rcd_quotas``);
``Context`` wraps ``rcd_create`` / ``rcd_destroy``.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Dict, Optional, Sequence, Tuple

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "librcd.so")

RCD_FEAT_I8 = 0
RCD_FEAT_BF16 = 1
RCD_SIM_DOT = 0
RCD_SIM_GAUSSIAN = 1
RCD_OBJ_FACILITY = 0
RCD_OBJ_GRAPH_CUT = 1

STATUS_NAMES = {0: "RCD_OK", 1: "RCD_ERR_INVALID_ARG", 2: "RCD_ERR_UNSUPPORTED", 3: "RCD_ERR_WORKSPACE_TOO_SMALL",
                4: "RCD_ERR_CUDA", 5: "RCD_ERR_TIMEOUT", 6: "RCD_ERR_INTERNAL"}

# every symbol include/rcd.h declares
EXPORTS = ["rcd_create", "rcd_destroy", "rcd_last_error", "rcd_version", "rcd_sync_status", "rcd_selftest_bounded_wait", "rcd_get_profile",
           "rcd_quotas", "rcd_similarity", "rcd_similarity_gaussian_workspace_bytes", "rcd_similarity_gaussian",
           "rcd_partition_workspace_bytes", "rcd_partition",
           "rcd_partition_host_workspace_bytes", "rcd_partition_host", "rcd_objective_workspace_bytes",
           "rcd_objective", "rcd_objective_class_static",
           "rcd_worker_lists_workspace_bytes", "rcd_worker_lists", "rcd_batch_sizes", "rcd_batch_sizes_rule",
           "rcd_yardstick_read", "rcd_yardstick_mma"]


class RcdError(RuntimeError):
    def __init__(self, status: int, message: str = ""):
        self.status = int(status)
        super().__init__("%s%s" % (STATUS_NAMES.get(self.status, str(status)), (": " + message) if message else ""))


class RcdConfig(C.Structure):
    _fields_ = [("sweep_batch_max", C.c_int32), ("similarity_path", C.c_int32), ("profile", C.c_int32),
                ("greedy_path", C.c_int32), ("similarity_kind", C.c_int32), ("objective", C.c_int32), ("sweep_mode", C.c_int32), ("async_group", C.c_int32),
                ("async_help_min", C.c_int32), ("threshold_from", C.c_int32), ("threshold_hit_shift", C.c_int32),
                ("lazy_mode", C.c_int32), ("lazy_from", C.c_int32), ("dense_ring", C.c_int32), ("incremental", C.c_int32), ("incremental_max", C.c_int32)]


class RcdProfile(C.Structure):
    _fields_ = [("total_ms", C.c_double), ("group_ms", C.c_double), ("similarity_ms", C.c_double),
                ("greedy_ms", C.c_double), ("sweep_ms", C.c_double), ("sweep_launches", C.c_int64),
                ("sweep_bytes", C.c_int64), ("sweep_elem_ops", C.c_int64), ("kernel_launches", C.c_int64),
                ("steps", C.c_int64), ("similarity_tc_launches", C.c_int64), ("persistent_sweep_ns", C.c_int64),
                ("persistent_pick_ns", C.c_int64), ("threshold_hits", C.c_int64),
                ("threshold_elems", C.c_int64), ("threshold_max_blocks", C.c_int64),
                ("async_lull_ns", C.c_int64), ("async_visits", C.c_int64), ("async_attempts", C.c_int64),
                ("lazy_sweeps", C.c_int64), ("lazy_misses", C.c_int64), ("lazy_rows", C.c_int64),
                ("lazy_rows_skipped", C.c_int64), ("incremental_updates", C.c_int64), ("incremental_rows", C.c_int64), ("threshold_pass_ns", C.c_int64), ("threshold_pass_bytes", C.c_int64), ("noted_picks", C.c_int64)]


def _load() -> C.CDLL:
    if not os.path.exists(LIB_PATH):
        raise ImportError("%s is missing: build it with `python -m paper_2211_00839_b200.build` "
                          "(there is no CPU fallback)" % LIB_PATH)
    lib = C.CDLL(LIB_PATH)
    vp, i64, i32, sz = C.c_void_p, C.c_int64, C.c_int32, C.c_size_t
    lib.rcd_create.argtypes = [C.POINTER(vp), C.c_int, C.POINTER(RcdConfig)]
    lib.rcd_destroy.argtypes = [vp]
    lib.rcd_destroy.restype = None
    lib.rcd_last_error.argtypes = [vp]
    lib.rcd_last_error.restype = C.c_char_p
    lib.rcd_version.argtypes = []
    lib.rcd_version.restype = C.c_char_p
    lib.rcd_sync_status.argtypes = [vp, vp]
    lib.rcd_selftest_bounded_wait.argtypes = [vp, vp]
    lib.rcd_get_profile.argtypes = [vp, C.POINTER(RcdProfile)]
    lib.rcd_quotas.argtypes = [i64, vp, i32, vp]
    lib.rcd_similarity.argtypes = [vp, vp, C.c_int, i64, i64, i64, vp, i64, vp]
    lib.rcd_similarity_gaussian_workspace_bytes.argtypes = [vp, i64, i64, C.POINTER(sz)]
    lib.rcd_similarity_gaussian.argtypes = [vp, vp, C.c_int, i64, i64, i64, vp, i64, vp, vp, sz, vp]
    for name in ("rcd_partition_workspace_bytes", "rcd_partition_host_workspace_bytes",
                 "rcd_objective_workspace_bytes"):
        getattr(lib, name).argtypes = [vp, C.c_int, i64, i64, i32, i64, i32, C.POINTER(sz)]
    lib.rcd_partition.argtypes = [vp, vp, C.c_int, i64, i64, vp, i32, vp, i32, vp, vp, vp, vp, sz, vp]
    lib.rcd_partition_host.argtypes = [vp, vp, C.c_int, i64, i64, vp, i32, vp, i32, vp, vp, vp, vp, sz, vp]
    lib.rcd_objective.argtypes = [vp, vp, C.c_int, i64, i64, vp, i32, vp, i32, vp, vp, vp, sz, vp]
    lib.rcd_objective_class_static.argtypes = [vp, vp, C.c_int, i64, i64, vp, i32, vp, vp, vp]
    lib.rcd_worker_lists_workspace_bytes.argtypes = [vp, i64, i32, C.POINTER(sz)]
    lib.rcd_worker_lists.argtypes = [vp, vp, i64, i32, vp, vp, vp, sz, vp]
    lib.rcd_batch_sizes.argtypes = [i64, vp, i32, vp]
    lib.rcd_batch_sizes_rule.argtypes = [i64, vp, i32, C.c_int, vp]
    lib.rcd_yardstick_read.argtypes = [vp, vp, sz, i32, vp]
    lib.rcd_yardstick_mma.argtypes = [vp, C.c_int, i32, C.POINTER(C.c_double), vp]
    for name in EXPORTS:
        f = getattr(lib, name)
        if name not in ("rcd_destroy", "rcd_last_error", "rcd_version"):
            f.restype = C.c_int
    return lib


lib = _load()


def rcd_version() -> str:
    return lib.rcd_version().decode()


def rcd_quotas(M: int, capacities: Sequence[float]) -> np.ndarray:
    """Integer quotas of one class (host only; no GPU needed)."""
    r = np.ascontiguousarray(capacities, dtype=np.float64)
    out = np.empty(len(r), dtype=np.int32)
    st = lib.rcd_quotas(int(M), r.ctypes.data_as(C.c_void_p), len(r), out.ctypes.data_as(C.c_void_p))
    if st != 0:
        raise RcdError(st, "rcd_quotas")
    return out


RCD_BATCH_PROPORTIONAL = 0
RCD_BATCH_AS_PRINTED = 1


def rcd_batch_sizes(B: int, capacities: Sequence[float], rule: int = RCD_BATCH_PROPORTIONAL) -> np.ndarray:
    """Per-worker batch sizes (host only; no GPU needed): b_j = B r_j / r_1, or with
    ``rule=RCD_BATCH_AS_PRINTED`` the ratio as Algorithm 2 prints it, B r_1 / r_j."""
    r = np.ascontiguousarray(capacities, dtype=np.float64)
    out = np.empty(len(r), dtype=np.int64)
    if rule == RCD_BATCH_PROPORTIONAL:
        st = lib.rcd_batch_sizes(int(B), r.ctypes.data_as(C.c_void_p), len(r), out.ctypes.data_as(C.c_void_p))
    else:
        st = lib.rcd_batch_sizes_rule(int(B), r.ctypes.data_as(C.c_void_p), len(r), int(rule), out.ctypes.data_as(C.c_void_p))
    if st != 0:
        raise RcdError(st, "rcd_batch_sizes")
    return out


def _torch():
    import torch
    return torch


def _dtype_code(t) -> int:
    torch = _torch()
    if t.dtype == torch.int8:
        return RCD_FEAT_I8
    if t.dtype == torch.bfloat16:
        return RCD_FEAT_BF16
    raise TypeError("features must be torch.int8 or torch.bfloat16, got %s" % t.dtype)


def features_to_torch(features: np.ndarray, device=None, pin: bool = False):
    """numpy int8, or uint16 bf16 bit patterns -> torch int8 / bfloat16 tensor (optionally pinned / on device)."""
    torch = _torch()
    if features.dtype == np.int8:
        t = torch.from_numpy(np.ascontiguousarray(features))
    elif features.dtype == np.uint16:
        t = torch.from_numpy(np.ascontiguousarray(features).view(np.int16)).view(torch.bfloat16)
    else:
        raise TypeError("features must be int8 or uint16 (bf16 bits)")
    if pin:
        t = t.pin_memory()
    if device is not None:
        t = t.to(device)
    return t


class Context:
    """Owns one ``rcd_ctx`` on a CUDA device."""

    def __init__(self, device: int = 0, sweep_batch_max: int = 0, similarity_path: int = 0, profile: int = 0,
                 greedy_path: int = 0, similarity_kind: int = 0, objective: int = 0, sweep_mode: int = 0,
                 async_group: int = 0, async_help_min: int = 0, threshold_from: int = 0, threshold_hit_shift: int = 0,
                 lazy_mode: int = 0, lazy_from: int = 0, dense_ring: int = 0, incremental: int = 0, incremental_max: int = 0):
        torch = _torch()
        if not torch.cuda.is_available():
            raise RcdError(4, "no CUDA device: this library has no CPU path")
        self.device = int(device)
        self.torch_device = torch.device("cuda", self.device)
        cfg = RcdConfig()
        cfg.sweep_batch_max = sweep_batch_max
        cfg.similarity_path = similarity_path
        cfg.profile = profile
        cfg.greedy_path = greedy_path
        cfg.similarity_kind = similarity_kind
        cfg.objective = objective
        cfg.sweep_mode = sweep_mode
        cfg.async_group = async_group
        cfg.async_help_min = async_help_min
        cfg.threshold_from = threshold_from
        cfg.threshold_hit_shift = threshold_hit_shift
        cfg.lazy_mode = lazy_mode
        cfg.lazy_from = lazy_from
        cfg.dense_ring = dense_ring
        cfg.incremental = incremental
        cfg.incremental_max = incremental_max
        self.similarity_kind = similarity_kind
        self._h = C.c_void_p()
        st = lib.rcd_create(C.byref(self._h), self.device, C.byref(cfg))
        if st != 0:
            raise RcdError(st, "rcd_create")
        self._ws = None

    def close(self):
        if getattr(self, "_h", None) is not None and self._h:
            lib.rcd_destroy(self._h)
            self._h = C.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def __enter__(self):
        return self

    def __exit__(self, *a):
        self.close()

    # -- helpers
    def _check(self, st: int):
        if st != 0:
            raise RcdError(st, lib.rcd_last_error(self._h).decode())

    def _stream(self):
        return C.c_void_p(_torch().cuda.current_stream(self.torch_device).cuda_stream)

    def workspace(self, nbytes: int):
        """A cached uint8 device tensor of at least ``nbytes`` (torch's allocator aligns it to 512 bytes)."""
        torch = _torch()
        if self._ws is None or self._ws.numel() < nbytes:
            self._ws = None
            self._ws = torch.empty(int(nbytes), dtype=torch.uint8, device=self.torch_device)
        return self._ws

    def selftest_bounded_wait(self):
        """Enqueue the wait that can never be satisfied; the following sync_status() raises RCD_ERR_TIMEOUT."""
        self._check(lib.rcd_selftest_bounded_wait(self._h, self._stream()))

    def sync_status(self):
        self._check(lib.rcd_sync_status(self._h, self._stream()))

    def profile(self) -> Dict[str, float]:
        p = RcdProfile()
        self._check(lib.rcd_get_profile(self._h, C.byref(p)))
        return {k: getattr(p, k) for k, _ in RcdProfile._fields_ if k != "reserved"}

    # -- entry points
    def rcd_similarity(self, X):
        """X: [batch, M, d] (or [M, d]) int8 / bfloat16 on the device -> S [batch, M, ld] int32 / float32."""
        torch = _torch()
        if X.dim() == 2:
            X = X.unsqueeze(0)
        X = X.contiguous()
        batch, M, d = X.shape
        ld = (M + 3) // 4 * 4
        code = _dtype_code(X)
        S = torch.empty((batch, M, ld), dtype=torch.int32 if code == RCD_FEAT_I8 else torch.float32,
                        device=X.device)
        self._check(lib.rcd_similarity(self._h, C.c_void_p(X.data_ptr()), code, M, d, batch,
                                       C.c_void_p(S.data_ptr()), ld, self._stream()))
        return S

    def _value_dtype(self, code: int):
        torch = _torch()
        return torch.int64 if (code == RCD_FEAT_I8 and self.similarity_kind == RCD_SIM_DOT) else torch.float64

    def rcd_similarity_gaussian(self, X):
        """X: [batch, M, d] (or [M, d]) int8 / bfloat16 on the device -> (S [batch, M, ld] float32, sigma [batch] float32)."""
        torch = _torch()
        if X.dim() == 2:
            X = X.unsqueeze(0)
        X = X.contiguous()
        batch, M, d = X.shape
        ld = (M + 3) // 4 * 4
        code = _dtype_code(X)
        S = torch.empty((batch, M, ld), dtype=torch.float32, device=X.device)
        sigma = torch.empty(batch, dtype=torch.float32, device=X.device)
        need = C.c_size_t()
        self._check(lib.rcd_similarity_gaussian_workspace_bytes(self._h, M, batch, C.byref(need)))
        ws = self.workspace(int(need.value))
        self._check(lib.rcd_similarity_gaussian(self._h, C.c_void_p(X.data_ptr()), code, M, d, batch,
                                                C.c_void_p(S.data_ptr()), ld, C.c_void_p(sigma.data_ptr()),
                                                C.c_void_p(ws.data_ptr()), ws.numel(), self._stream()))
        return S, sigma

    def partition_workspace_bytes(self, code: int, N: int, d: int, L: int, M_max: int, W: int, host: bool = False) -> int:
        out = C.c_size_t()
        fn = lib.rcd_partition_host_workspace_bytes if host else lib.rcd_partition_workspace_bytes
        self._check(fn(self._h, code, N, d, L, M_max, W, C.byref(out)))
        return int(out.value)

    def rcd_partition(self, features, labels, capacities: Sequence[float], L: int, M_max: Optional[int] = None,
                      want_order: bool = True, want_values: bool = True):
        """Device tensors in, device tensors out: (assignment[N] int32, order[N] int32 | None, part_values[L,W] | None).

        Enqueues on the current torch stream; call ``sync_status()`` (or synchronise) before reading."""
        torch = _torch()
        features = features.contiguous()
        labels = labels.contiguous()
        assert labels.dtype == torch.int32 and labels.is_cuda and features.is_cuda
        N, d = features.shape
        code = _dtype_code(features)
        caps = np.ascontiguousarray(capacities, dtype=np.float64)
        W = len(caps)
        if M_max is None:
            M_max = N
        nbytes = self.partition_workspace_bytes(code, N, d, L, M_max, W)
        ws = self.workspace(nbytes)
        assignment = torch.empty(N, dtype=torch.int32, device=features.device)
        order = torch.empty(N, dtype=torch.int32, device=features.device) if want_order else None
        values = None
        if want_values:
            values = torch.empty((L, W), dtype=self._value_dtype(code), device=features.device)
        self._check(lib.rcd_partition(self._h, C.c_void_p(features.data_ptr()), code, N, d,
                                      C.c_void_p(labels.data_ptr()), L, caps.ctypes.data_as(C.c_void_p), W,
                                      C.c_void_p(assignment.data_ptr()),
                                      C.c_void_p(order.data_ptr()) if order is not None else None,
                                      C.c_void_p(values.data_ptr()) if values is not None else None,
                                      C.c_void_p(ws.data_ptr()), ws.numel(), self._stream()))
        return assignment, order, values

    def rcd_partition_host(self, features, labels, capacities: Sequence[float], L: int, M_max: Optional[int] = None,
                           out: Optional[Tuple] = None):
        """Host tensors in (torch CPU tensors, ideally pinned), host tensors out; copies run inside the call.

        Returns (assignment[N] int32, order[N] int32, part_values[L,W]) as torch CPU tensors (pinned)."""
        torch = _torch()
        assert not features.is_cuda and not labels.is_cuda and labels.dtype == torch.int32
        features = features.contiguous()
        labels = labels.contiguous()
        N, d = features.shape
        code = _dtype_code(features)
        caps = np.ascontiguousarray(capacities, dtype=np.float64)
        W = len(caps)
        if M_max is None:
            M_max = N
        nbytes = self.partition_workspace_bytes(code, N, d, L, M_max, W, host=True)
        ws = self.workspace(nbytes)
        if out is None:
            assignment = torch.empty(N, dtype=torch.int32).pin_memory()
            order = torch.empty(N, dtype=torch.int32).pin_memory()
            values = torch.empty((L, W), dtype=self._value_dtype(code)).pin_memory()
        else:
            assignment, order, values = out
        with torch.cuda.device(self.torch_device):
            self._check(lib.rcd_partition_host(self._h, C.c_void_p(features.data_ptr()), code, N, d,
                                               C.c_void_p(labels.data_ptr()), L, caps.ctypes.data_as(C.c_void_p), W,
                                               C.c_void_p(assignment.data_ptr()), C.c_void_p(order.data_ptr()),
                                               C.c_void_p(values.data_ptr()), C.c_void_p(ws.data_ptr()), ws.numel(),
                                               self._stream()))
        return assignment, order, values

    def rcd_objective(self, features, labels, assignment, W: int, L: int, M_max: Optional[int] = None):
        """f(A_j^l) from the plain definition for a given assignment -> (part_values[L,W], total[1])."""
        torch = _torch()
        features = features.contiguous()
        labels = labels.contiguous()
        assignment = assignment.contiguous()
        N, d = features.shape
        code = _dtype_code(features)
        if M_max is None:
            M_max = N
        out = C.c_size_t()
        self._check(lib.rcd_objective_workspace_bytes(self._h, code, N, d, L, M_max, W, C.byref(out)))
        ws = self.workspace(int(out.value))
        vdt = self._value_dtype(code)
        values = torch.empty((L, W), dtype=vdt, device=features.device)
        total = torch.empty(1, dtype=vdt, device=features.device)
        self._check(lib.rcd_objective(self._h, C.c_void_p(features.data_ptr()), code, N, d,
                                      C.c_void_p(labels.data_ptr()), L, C.c_void_p(assignment.data_ptr()), W,
                                      C.c_void_p(values.data_ptr()), C.c_void_p(total.data_ptr()),
                                      C.c_void_p(ws.data_ptr()), ws.numel(), self._stream()))
        return values, total


def rcd_worker_lists(ctx: Context, assignment, W: int):
    """assignment [N] int32 on the device -> (offsets [W+1] int64, indices [N] int32): worker j's samples are
    indices[offsets[j]:offsets[j+1]], ascending."""
    torch = _torch()
    assignment = assignment.contiguous()
    N = assignment.numel()
    out = C.c_size_t()
    ctx._check(lib.rcd_worker_lists_workspace_bytes(ctx._h, N, W, C.byref(out)))
    ws = ctx.workspace(int(out.value))
    offsets = torch.empty(W + 1, dtype=torch.int64, device=assignment.device)
    indices = torch.empty(N, dtype=torch.int32, device=assignment.device)
    ctx._check(lib.rcd_worker_lists(ctx._h, C.c_void_p(assignment.data_ptr()), N, W, C.c_void_p(offsets.data_ptr()),
                                    C.c_void_p(indices.data_ptr()), C.c_void_p(ws.data_ptr()), ws.numel(), ctx._stream()))
    return offsets, indices


def rcd_objective_class_static(ctx: Context, S, assignment, W: int, part_values, total):
    """Block values of one class from its similarity matrix, for callers that cannot allocate.

    Everything is passed in: ``S`` [M, ld] int32 / float32, ``assignment`` [M] int32, and the
    outputs ``part_values`` [W] and ``total`` [1] (int64 for int32 S, float64 for float32 S), all
    device tensors the caller already owns.  This wrapper allocates nothing either."""
    torch = _torch()
    M, ld = S.shape
    code = RCD_FEAT_I8 if S.dtype == torch.int32 else RCD_FEAT_BF16
    ctx._check(lib.rcd_objective_class_static(ctx._h, C.c_void_p(S.data_ptr()), code, M, ld,
                                              C.c_void_p(assignment.data_ptr()), W,
                                              C.c_void_p(part_values.data_ptr()), C.c_void_p(total.data_ptr()),
                                              ctx._stream()))


def rcd_yardstick_read(ctx: Context, buffer, repeats: int = 1) -> int:
    """Enqueues the read-only sweep over ``buffer`` (any device tensor); returns the bytes one call reads."""
    nbytes = buffer.numel() * buffer.element_size() // 16 * 16
    ctx._check(lib.rcd_yardstick_read(ctx._h, C.c_void_p(buffer.data_ptr()), nbytes, int(repeats), ctx._stream()))
    return nbytes * int(repeats)


def rcd_yardstick_mma(ctx: Context, dtype_code: int, iterations: int) -> float:
    """Enqueues the tensor-core peak loop; returns the arithmetic operations the launch performs."""
    ops = C.c_double()
    ctx._check(lib.rcd_yardstick_mma(ctx._h, int(dtype_code), int(iterations), C.byref(ops), ctx._stream()))
    return float(ops.value)


def rcd_similarity(ctx: Context, X):
    return ctx.rcd_similarity(X)


def rcd_partition(ctx: Context, features, labels, capacities, L, **kw):
    return ctx.rcd_partition(features, labels, capacities, L, **kw)


def rcd_partition_host(ctx: Context, features, labels, capacities, L, **kw):
    return ctx.rcd_partition_host(features, labels, capacities, L, **kw)


def rcd_objective(ctx: Context, features, labels, assignment, W, L, **kw):
    return ctx.rcd_objective(features, labels, assignment, W, L, **kw)
