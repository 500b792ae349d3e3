"""ctypes binding of the C ABI declared in include/wpsgd.h. Same names, argument marshalling only."""
from __future__ import annotations

import ctypes
import os
from typing import Optional, Tuple

import numpy as np

LOSS_HINGE, LOSS_LOGISTIC, LOSS_SQUARED = 0, 1, 2
LR_CONST, LR_INV_SQRT = 0, 1
X_F32, X_BF16 = 0, 1

_STATUS = {0: "OK", 1: "INVALID_ARG", 2: "ALLOC", 3: "CUDA", 4: "STATE", 5: "UNSUPPORTED", 6: "TIMEOUT"}

EXPORTED_SYMBOLS = [
    "wpsgd_create", "wpsgd_destroy", "wpsgd_set_option", "wpsgd_set_node_ids", "wpsgd_run", "wpsgd_continue", "wpsgd_run_csr",
    "wpsgd_combine", "wpsgd_combine_weighted", "wpsgd_last_chain_ms", "wpsgd_get_models", "wpsgd_set_models", "wpsgd_get_weights", "wpsgd_weights",
    "wpsgd_sample_indices", "wpsgd_objective", "wpsgd_objective_csr", "wpsgd_solve_host", "wpsgd_solve_static", "wpsgd_check", "wpsgd_launch_count",
    "wpsgd_last_error", "wpsgd_continue_csr", "wpsgd_validate_csr", "wpsgd_span_valid", "wpsgd_sample_indices_host",
    "wpsgd_check_static", "wpsgd_solve_host_csr",
]

_HERE = os.path.dirname(os.path.abspath(__file__))
_lib = None


class WpsgdError(RuntimeError):
    def __init__(self, status: int, where: str, message: str):
        self.status = status
        self.status_name = _STATUS.get(status, str(status))
        super().__init__(f"{where}: WPSGD_ERR_{self.status_name}: {message}")


def library_path() -> str:
    return os.path.join(_HERE, "libwpsgd.so")


def load_library() -> ctypes.CDLL:
    """Load libwpsgd.so built in-tree. Raises if it has not been built: there is no other path."""
    global _lib
    if _lib is not None:
        return _lib
    path = library_path()
    if not os.path.exists(path):
        raise RuntimeError(f"{path} is missing: build it with `python -m paper_1708_04801_b200.build` "
                           "(the WP-SGD kernels have no CPU fallback)")
    lib = ctypes.CDLL(path)
    vp, i32, i64, u64, f32, f64 = (ctypes.c_void_p, ctypes.c_int32, ctypes.c_int64, ctypes.c_uint64, ctypes.c_float,
                                   ctypes.c_double)
    ci = ctypes.c_int
    lib.wpsgd_create.argtypes = [ci, vp, i32, i64, ctypes.POINTER(vp)]
    lib.wpsgd_destroy.argtypes = [vp]
    lib.wpsgd_set_option.argtypes = [vp, ctypes.c_char_p, i64]
    lib.wpsgd_set_node_ids.argtypes = [vp, vp]
    lib.wpsgd_run.argtypes = [vp, vp, ci, i64, vp, vp, vp, f32, ci, f32, ci, u64, vp]
    lib.wpsgd_continue.argtypes = [vp, vp, ci, i64, vp, vp, vp]
    lib.wpsgd_run_csr.argtypes = [vp, vp, vp, vp, vp, vp, vp, f32, ci, f32, ci, u64, vp]
    lib.wpsgd_combine.argtypes = [vp, f64, vp]
    lib.wpsgd_combine_weighted.argtypes = [vp, vp, vp]
    lib.wpsgd_last_chain_ms.argtypes = [vp, ctypes.POINTER(f32)]
    lib.wpsgd_get_models.argtypes = [vp, vp]
    lib.wpsgd_set_models.argtypes = [vp, vp]
    lib.wpsgd_get_weights.argtypes = [vp, f64, vp, ctypes.POINTER(ci)]
    lib.wpsgd_weights.argtypes = [vp, i32, f32, ci, f32, f64, vp, ctypes.POINTER(ci), ctypes.POINTER(f64)]
    lib.wpsgd_sample_indices.argtypes = [vp, u64, i32, i64, i64, i64, vp]
    lib.wpsgd_objective.argtypes = [vp, vp, ci, i64, vp, i64, vp, f32, ci, vp]
    lib.wpsgd_objective_csr.argtypes = [vp, vp, vp, vp, vp, i64, vp, f32, ci, vp]
    lib.wpsgd_solve_host.argtypes = [vp, vp, ci, vp, vp, vp, f32, ci, f32, ci, u64, vp, f64, vp]
    lib.wpsgd_solve_static.argtypes = [ci, vp, vp, ci, i64, vp, vp, vp, i32, i64, f32, ci, f32, ci, u64, vp, f64, vp]
    lib.wpsgd_check.argtypes = [vp]
    lib.wpsgd_continue_csr.argtypes = [vp, vp, vp, vp, vp, vp, vp]
    lib.wpsgd_validate_csr.argtypes = [vp, vp, vp, i64, i64]
    lib.wpsgd_span_valid.argtypes = [vp, i32, f32, f32, f64, i64, ctypes.POINTER(f64), ctypes.POINTER(ci)]
    lib.wpsgd_sample_indices_host.argtypes = [u64, i32, i64, i64, i64, i32, vp]
    lib.wpsgd_check_static.argtypes = [ci, vp]
    lib.wpsgd_solve_host_csr.argtypes = [vp, vp, vp, vp, vp, vp, vp, f32, ci, f32, ci, u64, vp, f64, vp]
    lib.wpsgd_launch_count.argtypes = [vp]
    lib.wpsgd_launch_count.restype = i64
    lib.wpsgd_last_error.argtypes = [vp]
    lib.wpsgd_last_error.restype = ctypes.c_char_p
    for name in EXPORTED_SYMBOLS:
        if name not in ("wpsgd_launch_count", "wpsgd_last_error"):
            getattr(lib, name).restype = ci
    _lib = lib
    return lib


def _host_i64(a) -> np.ndarray:
    return np.ascontiguousarray(np.asarray(a, dtype=np.int64))


def weights(n_steps, eta0: float, sched: int, lam: float, r: float = 0.0) -> Tuple[np.ndarray, bool, float]:
    """wpsgd_weights: Eq. 6 / Eq. 8 weights for given step counts, the Eq. 7 / 9 flag, and sum_j r^{T_j}."""
    lib = load_library()
    n = _host_i64(n_steps)
    w = np.zeros(n.shape[0], dtype=np.float64)
    flag = ctypes.c_int(0)
    tot = ctypes.c_double(0.0)
    st = lib.wpsgd_weights(n.ctypes.data, n.shape[0], eta0, sched, lam, r, w.ctypes.data, ctypes.byref(flag),
                           ctypes.byref(tot))
    if st:
        raise WpsgdError(st, "wpsgd_weights", lib.wpsgd_last_error(None).decode())
    return w, bool(flag.value), float(tot.value)


def span_valid(n_steps, eta0: float, lam: float, span: int, r: float = 0.0) -> Tuple[bool, float]:
    """wpsgd_span_valid: the paper's condition for averaging every `span` fastest-node steps on an unbalanced
    system, (k / sum_j r^{T_j}) (1 - eta lambda)^span < 1. Returns (holds, left-hand side)."""
    lib = load_library()
    n = _host_i64(n_steps)
    lhs = ctypes.c_double(0.0)
    flag = ctypes.c_int(0)
    st = lib.wpsgd_span_valid(n.ctypes.data, n.shape[0], eta0, lam, r, int(span), ctypes.byref(lhs), ctypes.byref(flag))
    if st:
        raise WpsgdError(st, "wpsgd_span_valid", lib.wpsgd_last_error(None).decode())
    return bool(flag.value), float(lhs.value)


def sample_indices_host(seed: int, node: int, m: int, n_begin: int, count: int, sampling: int = 0) -> np.ndarray:
    """wpsgd_sample_indices_host: the sample stream of the chains, computed on the host by the library."""
    lib = load_library()
    out = np.zeros(max(count, 0), dtype=np.uint32)
    st = lib.wpsgd_sample_indices_host(seed, node, m, n_begin, count, sampling, out.ctypes.data if count > 0 else None)
    if st:
        raise WpsgdError(st, "wpsgd_sample_indices_host", lib.wpsgd_last_error(None).decode())
    return out


def check_static(device: int = 0, stream=None):
    """wpsgd_check_static: wait for the stream and read the status word of wpsgd_solve_static's built-in array."""
    import torch

    lib = load_library()
    if stream is None:
        stream = torch.cuda.current_stream(device)
    st = lib.wpsgd_check_static(int(device), ctypes.c_void_p(stream.cuda_stream))
    if st:
        raise WpsgdError(st, "wpsgd_check_static", lib.wpsgd_last_error(None).decode())


def _xtype(X) -> int:
    import torch

    if X.dtype == torch.float32:
        return X_F32
    if X.dtype == torch.bfloat16:
        return X_BF16
    raise TypeError(f"features must be float32 or bfloat16, got {X.dtype}")


def solve_static(X, y, shard_off, n_steps, eta0, sched, lam, loss, seed, w0=None, r: float = 0.0, out=None,
                 stream=None):
    """wpsgd_solve_static: chains plus combination on dense device tensors without a context and without
    any device allocation by the library (its working memory is an array built into the library).
    For callers that may not allocate; sizes are limited (see include/wpsgd.h). `out` should be given by
    such callers; when it is None this wrapper allocates it with torch for convenience."""
    import torch

    lib = load_library()
    if not X.is_cuda or X.dim() != 2 or X.stride(1) != 1:
        raise TypeError("X must be a 2-D row-major CUDA tensor")
    dev = X.device.index
    so, ns = _host_i64(shard_off), _host_i64(n_steps)
    k, d = ns.shape[0], X.shape[1]
    if so.shape[0] != k + 1:
        raise ValueError("shard_off must have k+1 entries")
    if out is None:
        out = torch.empty(d, dtype=torch.float32, device=X.device)
    if stream is None:
        stream = torch.cuda.current_stream(dev)
    st = lib.wpsgd_solve_static(dev, ctypes.c_void_p(stream.cuda_stream), ctypes.c_void_p(X.data_ptr()), _xtype(X),
                                X.stride(0), ctypes.c_void_p(y.data_ptr()), so.ctypes.data, ns.ctypes.data, k, d, eta0,
                                sched, lam, loss, seed, ctypes.c_void_p(w0.data_ptr()) if w0 is not None else None, r,
                                ctypes.c_void_p(out.data_ptr()))
    if st:
        raise WpsgdError(st, "wpsgd_solve_static", lib.wpsgd_last_error(None).decode())
    return out


class Context:
    """One wpsgd_ctx. Methods carry the names of the C entry points without the prefix."""

    def __init__(self, k: int, d: int, device: Optional[int] = None, stream=None):
        import torch

        self._lib = load_library()
        if device is None:
            device = torch.cuda.current_device()
        self.device = int(device)
        if stream is None:
            stream = torch.cuda.current_stream(self.device)
        self._stream = stream  # keep alive
        self.k, self.d = int(k), int(d)
        h = ctypes.c_void_p()
        st = self._lib.wpsgd_create(self.device, ctypes.c_void_p(stream.cuda_stream), self.k, self.d, ctypes.byref(h))
        if st:
            raise WpsgdError(st, "wpsgd_create", self._lib.wpsgd_last_error(None).decode())
        self._h = h

    # -- plumbing ---------------------------------------------------------------------------------------
    def _ck(self, st: int, where: str):
        if st:
            raise WpsgdError(st, where, self._lib.wpsgd_last_error(self._h).decode())

    def _dev(self, t, dtype=None, n=None):
        import torch

        if t is None:
            return None
        if not isinstance(t, torch.Tensor) or not t.is_cuda or t.device.index != self.device:
            raise TypeError("expected a CUDA tensor on the context's device")
        if not t.is_contiguous():
            raise TypeError("expected a contiguous tensor")
        if dtype is not None and t.dtype != dtype:
            raise TypeError(f"expected dtype {dtype}, got {t.dtype}")
        if n is not None and t.numel() < n:
            raise ValueError(f"tensor too small: {t.numel()} < {n}")
        return ctypes.c_void_p(t.data_ptr())

    def destroy(self):
        if getattr(self, "_h", None):
            self._lib.wpsgd_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.destroy()
        except Exception:
            pass

    def __enter__(self):
        return self

    def __exit__(self, *exc):
        self.destroy()

    # -- entry points -----------------------------------------------------------------------------------
    def set_option(self, name: str, value: int):
        self._ck(self._lib.wpsgd_set_option(self._h, name.encode(), int(value)), "wpsgd_set_option")

    def set_node_ids(self, ids=None):
        if ids is None:
            self._ck(self._lib.wpsgd_set_node_ids(self._h, None), "wpsgd_set_node_ids")
            return
        a = np.ascontiguousarray(np.asarray(ids, dtype=np.int32))
        if a.shape[0] != self.k:
            raise ValueError("ids must have k entries")
        self._ck(self._lib.wpsgd_set_node_ids(self._h, a.ctypes.data), "wpsgd_set_node_ids")

    def run(self, X, y, shard_off, n_steps, eta0, sched, lam, loss, seed, w0=None):
        import torch

        if X.dim() != 2 or X.stride(1) != 1:
            raise TypeError("X must be a 2-D row-major tensor")
        so, ns = _host_i64(shard_off), _host_i64(n_steps)
        if so.shape[0] != self.k + 1 or ns.shape[0] != self.k:
            raise ValueError("shard_off must have k+1 entries and n_steps k entries")
        xp = ctypes.c_void_p(X.data_ptr()) if X.is_cuda and X.device.index == self.device else None
        if xp is None:
            raise TypeError("X must live on the context's device")
        self._ck(self._lib.wpsgd_run(self._h, xp, _xtype(X), X.stride(0), self._dev(y, torch.float32, int(so[-1])),
                                     so.ctypes.data, ns.ctypes.data, eta0, sched, lam, loss, seed,
                                     self._dev(w0, torch.float32, self.d)), "wpsgd_run")

    def continue_(self, X, y, shard_off, n_more):
        import torch

        so, ns = _host_i64(shard_off), _host_i64(n_more)
        if so.shape[0] != self.k + 1 or ns.shape[0] != self.k:
            raise ValueError("shard_off must have k+1 entries and n_more k entries")
        self._ck(self._lib.wpsgd_continue(self._h, ctypes.c_void_p(X.data_ptr()), _xtype(X), X.stride(0),
                                          self._dev(y, torch.float32, int(so[-1])), so.ctypes.data, ns.ctypes.data),
                 "wpsgd_continue")

    def run_csr(self, row_ptr, col_idx, val, y, shard_off, n_steps, eta0, sched, lam, loss, seed, w0=None):
        import torch

        so, ns = _host_i64(shard_off), _host_i64(n_steps)
        if so.shape[0] != self.k + 1 or ns.shape[0] != self.k:
            raise ValueError("shard_off must have k+1 entries and n_steps k entries")
        self._ck(self._lib.wpsgd_run_csr(self._h, self._dev(row_ptr, torch.int64, int(so[-1]) + 1),
                                         self._dev(col_idx, torch.int32), self._dev(val, torch.float32),
                                         self._dev(y, torch.float32, int(so[-1])), so.ctypes.data, ns.ctypes.data,
                                         eta0, sched, lam, loss, seed, self._dev(w0, torch.float32, self.d)),
                 "wpsgd_run_csr")

    def continue_csr(self, row_ptr, col_idx, val, y, shard_off, n_more):
        import torch

        so, ns = _host_i64(shard_off), _host_i64(n_more)
        if so.shape[0] != self.k + 1 or ns.shape[0] != self.k:
            raise ValueError("shard_off must have k+1 entries and n_more k entries")
        self._ck(self._lib.wpsgd_continue_csr(self._h, self._dev(row_ptr, torch.int64, int(so[-1]) + 1),
                                              self._dev(col_idx, torch.int32), self._dev(val, torch.float32),
                                              self._dev(y, torch.float32, int(so[-1])), so.ctypes.data, ns.ctypes.data),
                 "wpsgd_continue_csr")

    def validate_csr(self, row_ptr, col_idx):
        import torch

        n_rows = int(row_ptr.numel()) - 1
        self._ck(self._lib.wpsgd_validate_csr(self._h, self._dev(row_ptr, torch.int64), self._dev(col_idx, torch.int32),
                                              n_rows, int(col_idx.numel())), "wpsgd_validate_csr")

    def run_workload(self, wl):
        """run / run_csr on a workload object (tensors already on the device)."""
        if wl.sparse:
            self.run_csr(wl.row_ptr, wl.col_idx, wl.val, wl.y, wl.shard_off, wl.n_steps, wl.eta0, wl.sched, wl.lam,
                         wl.loss, wl.seed, wl.w0)
        else:
            self.run(wl.X, wl.y, wl.shard_off, wl.n_steps, wl.eta0, wl.sched, wl.lam, wl.loss, wl.seed, wl.w0)

    def combine(self, r: float = 0.0, out=None):
        import torch

        if out is None:
            out = torch.empty(self.d, dtype=torch.float32, device=f"cuda:{self.device}")
        self._ck(self._lib.wpsgd_combine(self._h, r, self._dev(out, torch.float32, self.d)), "wpsgd_combine")
        return out

    def combine_weighted(self, weights, out=None):
        import torch

        w = np.ascontiguousarray(np.asarray(weights, dtype=np.float64))
        if w.shape[0] != self.k:
            raise ValueError("weights must have k entries")
        if out is None:
            out = torch.empty(self.d, dtype=torch.float32, device=f"cuda:{self.device}")
        self._ck(self._lib.wpsgd_combine_weighted(self._h, w.ctypes.data, self._dev(out, torch.float32, self.d)),
                 "wpsgd_combine_weighted")
        return out

    def last_chain_ms(self) -> float:
        ms = ctypes.c_float(0.0)
        self._ck(self._lib.wpsgd_last_chain_ms(self._h, ctypes.byref(ms)), "wpsgd_last_chain_ms")
        return float(ms.value)

    def get_models(self, out=None):
        import torch

        if out is None:
            out = torch.empty((self.k, self.d), dtype=torch.float32, device=f"cuda:{self.device}")
        self._ck(self._lib.wpsgd_get_models(self._h, self._dev(out, torch.float32, self.k * self.d)), "wpsgd_get_models")
        return out

    def set_models(self, v):
        import torch

        self._ck(self._lib.wpsgd_set_models(self._h, self._dev(v, torch.float32, self.d)), "wpsgd_set_models")

    def get_weights(self, r: float = 0.0):
        w = np.zeros(self.k, dtype=np.float64)
        flag = ctypes.c_int(0)
        self._ck(self._lib.wpsgd_get_weights(self._h, r, w.ctypes.data, ctypes.byref(flag)), "wpsgd_get_weights")
        return w, bool(flag.value)

    def sample_indices(self, seed: int, node: int, m: int, n_begin: int, count: int):
        import torch

        out = torch.empty(max(count, 0), dtype=torch.int32, device=f"cuda:{self.device}")
        self._ck(self._lib.wpsgd_sample_indices(self._h, seed, node, m, n_begin, count,
                                                ctypes.c_void_p(out.data_ptr()) if count > 0 else None),
                 "wpsgd_sample_indices")
        return out

    def objective(self, X, y, w, lam: float, loss: int):
        import torch

        out = torch.empty(2, dtype=torch.float64, device=f"cuda:{self.device}")
        self._ck(self._lib.wpsgd_objective(self._h, ctypes.c_void_p(X.data_ptr()), _xtype(X), X.stride(0),
                                           self._dev(y, torch.float32, X.shape[0]), X.shape[0],
                                           self._dev(w, torch.float32, self.d), lam, loss, self._dev(out)),
                 "wpsgd_objective")
        return out

    def objective_csr(self, row_ptr, col_idx, val, y, w, lam: float, loss: int):
        import torch

        out = torch.empty(2, dtype=torch.float64, device=f"cuda:{self.device}")
        n_rows = int(y.numel())
        self._ck(self._lib.wpsgd_objective_csr(self._h, self._dev(row_ptr, torch.int64, n_rows + 1),
                                               self._dev(col_idx, torch.int32), self._dev(val, torch.float32),
                                               self._dev(y, torch.float32), n_rows, self._dev(w, torch.float32, self.d),
                                               lam, loss, self._dev(out)), "wpsgd_objective_csr")
        return out

    def solve_host(self, X, y, shard_off, n_steps, eta0, sched, lam, loss, seed, w0=None, r: float = 0.0, out=None):
        """Host tensors in (ideally pinned), host tensor out; copies are part of the call."""
        import torch

        for t in (X, y) + ((w0,) if w0 is not None else ()):
            if t.is_cuda or not t.is_contiguous():
                raise TypeError("solve_host takes contiguous host tensors")
        so, ns = _host_i64(shard_off), _host_i64(n_steps)
        if out is None:
            out = torch.empty(self.d, dtype=torch.float32).pin_memory()
        self._ck(self._lib.wpsgd_solve_host(self._h, ctypes.c_void_p(X.data_ptr()), _xtype(X),
                                            ctypes.c_void_p(y.data_ptr()), so.ctypes.data, ns.ctypes.data, eta0, sched,
                                            lam, loss, seed, ctypes.c_void_p(w0.data_ptr()) if w0 is not None else None,
                                            r, ctypes.c_void_p(out.data_ptr())), "wpsgd_solve_host")
        return out

    def solve_host_csr(self, row_ptr, col_idx, val, y, shard_off, n_steps, eta0, sched, lam, loss, seed, w0=None,
                       r: float = 0.0, out=None):
        """Host CSR tensors in (ideally pinned), host tensor out; copies are part of the call."""
        import torch

        for t, dt in ((row_ptr, torch.int64), (col_idx, torch.int32), (val, torch.float32), (y, torch.float32)):
            if t.is_cuda or not t.is_contiguous() or t.dtype != dt:
                raise TypeError("solve_host_csr takes contiguous host tensors (int64 row_ptr, int32 col_idx, float32 val, y)")
        so, ns = _host_i64(shard_off), _host_i64(n_steps)
        if out is None:
            out = torch.empty(self.d, dtype=torch.float32).pin_memory()
        self._ck(self._lib.wpsgd_solve_host_csr(self._h, ctypes.c_void_p(row_ptr.data_ptr()), ctypes.c_void_p(col_idx.data_ptr()),
                                                ctypes.c_void_p(val.data_ptr()), ctypes.c_void_p(y.data_ptr()),
                                                so.ctypes.data, ns.ctypes.data, eta0, sched, lam, loss, seed,
                                                ctypes.c_void_p(w0.data_ptr()) if w0 is not None else None, r,
                                                ctypes.c_void_p(out.data_ptr())), "wpsgd_solve_host_csr")
        return out

    def check(self):
        self._ck(self._lib.wpsgd_check(self._h), "wpsgd_check")

    def launch_count(self) -> int:
        return int(self._lib.wpsgd_launch_count(self._h))
