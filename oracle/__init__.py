"""Python access to the WP-SGD CPU oracle (test infrastructure only).

The oracle itself is `wpsgd_oracle.cpp` (plain single-threaded C++, fp64 state). This
module compiles it with g++ on first use and exposes its functions on numpy arrays.
Only tests, the smoke check and the benchmark's CPU-baseline leg may import it; the
CUDA library and its Python binding never do.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
import threading

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "wpsgd_oracle.cpp")
_LIB = os.path.join(_HERE, "liboracle_wpsgd.so")
_lock = threading.Lock()
_lib = None

c_i64p = ctypes.POINTER(ctypes.c_int64)
c_f32p = ctypes.POINTER(ctypes.c_float)
c_f64p = ctypes.POINTER(ctypes.c_double)
c_u32p = ctypes.POINTER(ctypes.c_uint32)
c_i32p = ctypes.POINTER(ctypes.c_int32)


def build(force: bool = False) -> str:
    """Compile the oracle into a shared object next to its source (no fast-math, no FMA contraction)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".tmp{os.getpid()}"
        subprocess.check_call(["g++", "-O2", "-ffp-contract=off", "-fPIC", "-shared", "-std=c++17", _SRC, "-o", tmp])
        os.replace(tmp, _LIB)
    return _LIB


def lib() -> ctypes.CDLL:
    global _lib
    with _lock:
        if _lib is None:
            _lib = ctypes.CDLL(build())
            _lib.oracle_sample_indices.argtypes = [ctypes.c_uint64, ctypes.c_int32, ctypes.c_int64, ctypes.c_int64,
                                                   ctypes.c_int64, c_u32p]
            _lib.oracle_philox4x32_10.argtypes = [c_u32p, c_u32p, c_u32p]
            _lib.oracle_philox4x32_10.restype = None
            _lib.oracle_run_dense.argtypes = [ctypes.c_void_p, ctypes.c_int, ctypes.c_int64, c_f32p, c_i64p, c_i64p,
                                              ctypes.c_int32, ctypes.c_int64, ctypes.c_float, ctypes.c_int,
                                              ctypes.c_float, ctypes.c_int, ctypes.c_uint64, c_f32p, ctypes.c_int64,
                                              ctypes.c_int, c_f64p]
            for name in ("oracle_run_csr_literal", "oracle_run_csr_lazy"):
                fn = getattr(_lib, name)
                base = [c_i64p, c_i32p, c_f32p, c_f32p, c_i64p, c_i64p, ctypes.c_int32, ctypes.c_int64, ctypes.c_float,
                        ctypes.c_int, ctypes.c_float, ctypes.c_int, ctypes.c_uint64, c_f32p]
                fn.argtypes = base + ([ctypes.c_int32] if name.endswith("lazy") else []) + [c_f64p]
            _lib.oracle_weights.argtypes = [c_i64p, ctypes.c_int32, ctypes.c_float, ctypes.c_int, ctypes.c_float,
                                            ctypes.c_double, c_f64p, ctypes.POINTER(ctypes.c_int), c_f64p]
            _lib.oracle_combine.argtypes = [c_f64p, c_f64p, ctypes.c_int32, ctypes.c_int64, c_f64p]
            _lib.oracle_objective_dense.argtypes = [ctypes.c_void_p, ctypes.c_int, ctypes.c_int64, c_f32p,
                                                    ctypes.c_int64, ctypes.c_int64, c_f64p, ctypes.c_float,
                                                    ctypes.c_int, c_f64p, c_f64p]
            _lib.oracle_objective_csr.argtypes = [c_i64p, c_i32p, c_f32p, c_f32p, ctypes.c_int64, ctypes.c_int64, c_f64p,
                                                  ctypes.c_float, ctypes.c_int, c_f64p, c_f64p]
    return _lib


def _p(a, ty):
    return None if a is None else a.ctypes.data_as(ty)


def _np(a, dtype):
    """numpy view of a numpy array or CPU torch tensor, contiguous, of the given dtype."""
    if a is None:
        return None
    if hasattr(a, "detach"):
        a = a.detach().cpu().contiguous().numpy()
    a = np.ascontiguousarray(a)
    assert a.dtype == dtype, (a.dtype, dtype)
    return a


def set_sampling(mode: int):
    """0: i.i.d. uniform draws (default); 1: one fixed shuffle per node, cycled. Applies to later calls."""
    if lib().oracle_set_sampling(int(mode)):
        raise ValueError("unknown sampling mode")


def philox4x32_10(ctr, key):
    c = np.asarray(ctr, dtype=np.uint32)
    k = np.asarray(key, dtype=np.uint32)
    out = np.zeros(4, dtype=np.uint32)
    lib().oracle_philox4x32_10(_p(c, c_u32p), _p(k, c_u32p), _p(out, c_u32p))
    return out


def sample_indices(seed: int, node: int, m: int, n_begin: int, count: int) -> np.ndarray:
    out = np.zeros(count, dtype=np.uint32)
    rc = lib().oracle_sample_indices(seed, node, m, n_begin, count, _p(out, c_u32p))
    if rc:
        raise ValueError("oracle_sample_indices: invalid argument")
    return out


def _dense_ptr(X):
    """(pointer, xtype, ld, keepalive) for an fp32 numpy/torch matrix or a bf16 torch matrix."""
    if hasattr(X, "detach"):
        import torch

        X = X.detach().cpu().contiguous()
        if X.dtype == torch.bfloat16:
            raw = X.view(torch.int16).numpy()
            return raw.ctypes.data_as(ctypes.c_void_p), 1, X.shape[1], raw
        X = X.numpy()
    X = np.ascontiguousarray(X)
    assert X.dtype == np.float32
    return X.ctypes.data_as(ctypes.c_void_p), 0, X.shape[1], X


def run_dense(X, y, shard_off, n_steps, d, eta0, sched, lam, loss, seed, w0=None, step_begin=0, W_resume=None):
    """Per-node chains of Algorithm 1 on dense rows; returns W [k, d] float64."""
    ptr, xtype, ld, keep = _dense_ptr(X)
    y = _np(y, np.float32)
    so = _np(shard_off, np.int64)
    ns = _np(n_steps, np.int64)
    w0 = _np(w0, np.float32)
    k = ns.shape[0]
    if W_resume is not None:
        W = np.array(W_resume, dtype=np.float64, order="C", copy=True)
    else:
        W = np.zeros((k, d), dtype=np.float64)
    rc = lib().oracle_run_dense(ptr, xtype, ld, _p(y, c_f32p), _p(so, c_i64p), _p(ns, c_i64p), k, d, eta0, sched, lam,
                                loss, seed, _p(w0, c_f32p), step_begin, 1 if W_resume is not None else 0, _p(W, c_f64p))
    if rc:
        raise ValueError("oracle_run_dense: invalid argument")
    return W


def run_csr(row_ptr, col_idx, val, y, shard_off, n_steps, d, eta0, sched, lam, loss, seed, w0=None, literal=False,
            one_node=-1):
    """Per-node chains on CSR rows. literal=True: O(d)-per-step definition; else the scaled form."""
    rp = _np(row_ptr, np.int64)
    ci = _np(col_idx, np.int32)
    va = _np(val, np.float32)
    y = _np(y, np.float32)
    so = _np(shard_off, np.int64)
    ns = _np(n_steps, np.int64)
    w0 = _np(w0, np.float32)
    k = ns.shape[0]
    W = np.zeros((k, d) if one_node < 0 else (d,), dtype=np.float64)
    args = [_p(rp, c_i64p), _p(ci, c_i32p), _p(va, c_f32p), _p(y, c_f32p), _p(so, c_i64p), _p(ns, c_i64p), k, d, eta0,
            sched, lam, loss, seed, _p(w0, c_f32p)]
    if literal:
        assert one_node < 0
        rc = lib().oracle_run_csr_literal(*args, _p(W, c_f64p))
    else:
        rc = lib().oracle_run_csr_lazy(*args, one_node, _p(W, c_f64p))
    if rc:
        raise ValueError("oracle_run_csr: invalid argument")
    return W


def weights(n_steps, eta0, sched, lam, r=0.0):
    """(weights [k] float64, Eq.7/9 condition holds, sum_i r^{T_i})."""
    ns = _np(n_steps, np.int64)
    k = ns.shape[0]
    w = np.zeros(k, dtype=np.float64)
    flag = ctypes.c_int(0)
    tot = np.zeros(1, dtype=np.float64)
    rc = lib().oracle_weights(_p(ns, c_i64p), k, eta0, sched, lam, r, _p(w, c_f64p), ctypes.byref(flag), _p(tot, c_f64p))
    if rc:
        raise ValueError("oracle_weights: invalid argument")
    return w, bool(flag.value), float(tot[0])


def combine(W, wts):
    W = np.ascontiguousarray(W, dtype=np.float64)
    wts = np.ascontiguousarray(wts, dtype=np.float64)
    k, d = W.shape
    v = np.zeros(d, dtype=np.float64)
    lib().oracle_combine(_p(W, c_f64p), _p(wts, c_f64p), k, d, _p(v, c_f64p))
    return v


def objective_dense(X, y, w, lam, loss):
    ptr, xtype, ld, keep = _dense_ptr(X)
    y = _np(y, np.float32)
    w = np.ascontiguousarray(w, dtype=np.float64)
    obj = np.zeros(1)
    err = np.zeros(1)
    lib().oracle_objective_dense(ptr, xtype, ld, _p(y, c_f32p), y.shape[0], w.shape[0], _p(w, c_f64p), lam, loss,
                                 _p(obj, c_f64p), _p(err, c_f64p))
    return float(obj[0]), float(err[0])


def objective_csr(row_ptr, col_idx, val, y, w, lam, loss):
    rp, ci, va, y = _np(row_ptr, np.int64), _np(col_idx, np.int32), _np(val, np.float32), _np(y, np.float32)
    w = np.ascontiguousarray(w, dtype=np.float64)
    obj, err = np.zeros(1), np.zeros(1)
    lib().oracle_objective_csr(_p(rp, c_i64p), _p(ci, c_i32p), _p(va, c_f32p), _p(y, c_f32p), y.shape[0], w.shape[0],
                               _p(w, c_f64p), lam, loss, _p(obj, c_f64p), _p(err, c_f64p))
    return float(obj[0]), float(err[0])


def solve(wl, r=0.0):
    """Whole path on a workload object: chains then weighted combination. Returns (v, W, weights)."""
    if wl.sparse:
        W = run_csr(wl.row_ptr, wl.col_idx, wl.val, wl.y, wl.shard_off, wl.n_steps, wl.d, wl.eta0, wl.sched, wl.lam,
                    wl.loss, wl.seed, wl.w0)
    else:
        W = run_dense(wl.X, wl.y, wl.shard_off, wl.n_steps, wl.d, wl.eta0, wl.sched, wl.lam, wl.loss, wl.seed, wl.w0)
    wts, _, _ = weights(wl.n_steps, wl.eta0, wl.sched, wl.lam, r)
    return combine(W, wts), W, wts
