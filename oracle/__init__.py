"""ctypes access to the fp64 CPU oracle (attention by the plain definition; planner by brute force).

TEST INFRASTRUCTURE ONLY: the tests, the smoke check and the benchmark's CPU-baseline leg may
import this package; the product package never does.  It imports nothing from the product.

The C sources beside this file are compiled with gcc (OpenMP) into ``liboracle.so`` on first
use, and again whenever a source is newer than the library.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
import threading

import numpy as np

_DIR = os.path.dirname(os.path.abspath(__file__))
_SOURCES = [os.path.join(_DIR, "attn_oracle.c"), os.path.join(_DIR, "plan_oracle.c"),
            os.path.join(_DIR, "inter_oracle.c")]
_LIB_PATH = os.path.join(_DIR, "liboracle.so")
_lock = threading.Lock()
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle if the library is missing or older than its sources."""
    stale = force or not os.path.exists(_LIB_PATH) or any(
        os.path.getmtime(s) > os.path.getmtime(_LIB_PATH) for s in _SOURCES)
    if stale:
        tmp = _LIB_PATH + f".tmp{os.getpid()}"
        cmd = ["gcc", "-O3", "-fopenmp", "-fPIC", "-shared", "-std=gnu11", "-Wall",
               "-o", tmp, *_SOURCES, "-lm"]
        subprocess.run(cmd, check=True)
        os.replace(tmp, _LIB_PATH)
    return _LIB_PATH


class PlanParams(ctypes.Structure):
    _fields_ = [("n_heads", ctypes.c_int32), ("head_dim", ctypes.c_int32),
                ("elt_bytes", ctypes.c_int32), ("n_layers", ctypes.c_int32),
                ("const_bytes", ctypes.c_int64), ("fixed_cost", ctypes.c_int64)]


def _load():
    global _lib
    with _lock:
        if _lib is None:
            lib = ctypes.CDLL(build())
            u16p = ctypes.POINTER(ctypes.c_uint16)
            i32p = ctypes.POINTER(ctypes.c_int32)
            f64p = ctypes.POINTER(ctypes.c_double)
            ci, cd = ctypes.c_int, ctypes.c_double
            lib.oracle_num_threads.restype = ci
            lib.oracle_attn_fwd.argtypes = [u16p, u16p, u16p, i32p, ci, ci, ci, ci, cd, f64p, f64p]
            lib.oracle_attn_bwd.argtypes = [u16p, u16p, u16p, u16p, i32p, ci, ci, ci, ci, cd,
                                            f64p, f64p, f64p]
            lib.oracle_attn_rows.argtypes = [u16p, u16p, u16p, u16p, i32p, ci, ci, ci, cd, ci, ci,
                                             ci, i32p, f64p, f64p, f64p]
            lib.oracle_attn_cols.argtypes = [u16p, u16p, u16p, u16p, i32p, ci, ci, ci, cd, ci, ci,
                                             ci, i32p, f64p, f64p]
            lib.oracle_plan_bruteforce_weighted.argtypes = [
                i32p, ctypes.POINTER(ctypes.c_int64), ctypes.c_int32, ctypes.c_int64, ctypes.POINTER(PlanParams),
                i32p, i32p, i32p, ctypes.POINTER(ctypes.c_uint64), ctypes.POINTER(ctypes.c_uint64)]
            lib.oracle_inter_bruteforce.argtypes = [
                ctypes.POINTER(ctypes.c_int64), ctypes.c_int32, ctypes.c_int32, ctypes.c_int32, i32p,
                ctypes.POINTER(ctypes.c_uint64), ctypes.POINTER(ctypes.c_uint64)]
            _lib = lib
    return _lib


def num_threads() -> int:
    return int(_load().oracle_num_threads())


def _bits(x, shape=None) -> np.ndarray:
    """bf16 bit patterns as a contiguous uint16 array.  Accepts uint16 numpy arrays or torch
    bfloat16 CPU tensors."""
    if hasattr(x, "dtype") and str(x.dtype) == "torch.bfloat16":
        import torch
        x = x.detach().cpu().contiguous().view(torch.int16).numpy().view(np.uint16)
    x = np.ascontiguousarray(x)
    if x.dtype != np.uint16:
        raise TypeError("oracle inputs are bf16 bit patterns (uint16) or torch.bfloat16 tensors")
    if shape is not None and tuple(x.shape) != tuple(shape):
        raise ValueError(f"expected shape {shape}, got {x.shape}")
    return x


def _p(a, ct):
    return a.ctypes.data_as(ctypes.POINTER(ct))


def _cu(cu_seqlens) -> np.ndarray:
    cu = np.ascontiguousarray(np.asarray(cu_seqlens), dtype=np.int32)
    if cu.ndim != 1 or cu.size < 1 or cu[0] != 0 or np.any(np.diff(cu) < 0):
        raise ValueError("cu_seqlens must start at 0 and be non-decreasing")
    return cu


def _scale(scale, d):
    return float(scale) if scale else 1.0 / float(np.sqrt(np.float64(d)))


def attn_fwd(q, k, v, cu_seqlens, causal: bool, scale: float = 0.0):
    """O [T,H,d] and lse [H,T] in float64 for bf16 q, k, v of shape [T,H,d]."""
    q = _bits(q)
    T, H, d = q.shape
    k, v, cu = _bits(k, q.shape), _bits(v, q.shape), _cu(cu_seqlens)
    if cu[-1] != T:
        raise ValueError("cu_seqlens[-1] must equal the token count")
    O = np.zeros((T, H, d), np.float64)
    lse = np.zeros((H, T), np.float64)
    rc = _load().oracle_attn_fwd(_p(q, ctypes.c_uint16), _p(k, ctypes.c_uint16), _p(v, ctypes.c_uint16),
                                 _p(cu, ctypes.c_int32), cu.size - 1, H, d, int(bool(causal)),
                                 _scale(scale, d), _p(O, ctypes.c_double), _p(lse, ctypes.c_double))
    if rc:
        raise RuntimeError(f"oracle_attn_fwd failed ({rc})")
    return O, lse


def attn_bwd(q, k, v, d_o, cu_seqlens, causal: bool, scale: float = 0.0):
    """dQ, dK, dV [T,H,d] in float64 for the loss sum(O * dO)."""
    q = _bits(q)
    T, H, d = q.shape
    k, v, g, cu = _bits(k, q.shape), _bits(v, q.shape), _bits(d_o, q.shape), _cu(cu_seqlens)
    if cu[-1] != T:
        raise ValueError("cu_seqlens[-1] must equal the token count")
    dq, dk, dv = (np.zeros((T, H, d), np.float64) for _ in range(3))
    u16 = ctypes.c_uint16
    rc = _load().oracle_attn_bwd(_p(q, u16), _p(k, u16), _p(v, u16), _p(g, u16), _p(cu, ctypes.c_int32),
                                 cu.size - 1, H, d, int(bool(causal)), _scale(scale, d),
                                 _p(dq, ctypes.c_double), _p(dk, ctypes.c_double), _p(dv, ctypes.c_double))
    if rc:
        raise RuntimeError(f"oracle_attn_bwd failed ({rc})")
    return dq, dk, dv


def attn_rows(q, k, v, d_o, cu_seqlens, causal: bool, seq: int, head: int, rows, scale: float = 0.0):
    """(O_rows [n,d], lse_rows [n], dQ_rows [n,d] or None) for the given rows (relative to the
    sequence start) of one (sequence, head).  Pass d_o=None to skip dQ."""
    q = _bits(q)
    T, H, d = q.shape
    k, v, cu = _bits(k, q.shape), _bits(v, q.shape), _cu(cu_seqlens)
    g = _bits(d_o, q.shape) if d_o is not None else None
    rows = np.ascontiguousarray(rows, dtype=np.int32)
    n = rows.size
    O = np.zeros((n, d), np.float64)
    lse = np.zeros((n,), np.float64)
    dq = np.zeros((n, d), np.float64) if g is not None else None
    u16 = ctypes.c_uint16
    rc = _load().oracle_attn_rows(_p(q, u16), _p(k, u16), _p(v, u16), _p(g, u16) if g is not None else None,
                                  _p(cu, ctypes.c_int32), H, d, int(bool(causal)), _scale(scale, d),
                                  int(seq), int(head), n, _p(rows, ctypes.c_int32), _p(O, ctypes.c_double),
                                  _p(lse, ctypes.c_double),
                                  _p(dq, ctypes.c_double) if dq is not None else None)
    if rc:
        raise RuntimeError(f"oracle_attn_rows failed ({rc})")
    return O, lse, dq


def attn_cols(q, k, v, d_o, cu_seqlens, causal: bool, seq: int, head: int, cols, scale: float = 0.0):
    """(dK_cols [n,d], dV_cols [n,d]) for the given key columns of one (sequence, head)."""
    q = _bits(q)
    T, H, d = q.shape
    k, v, g, cu = _bits(k, q.shape), _bits(v, q.shape), _bits(d_o, q.shape), _cu(cu_seqlens)
    cols = np.ascontiguousarray(cols, dtype=np.int32)
    n = cols.size
    dk = np.zeros((n, d), np.float64)
    dv = np.zeros((n, d), np.float64)
    u16 = ctypes.c_uint16
    rc = _load().oracle_attn_cols(_p(q, u16), _p(k, u16), _p(v, u16), _p(g, u16), _p(cu, ctypes.c_int32),
                                  H, d, int(bool(causal)), _scale(scale, d), int(seq), int(head), n,
                                  _p(cols, ctypes.c_int32), _p(dk, ctypes.c_double), _p(dv, ctypes.c_double))
    if rc:
        raise RuntimeError(f"oracle_attn_cols failed ({rc})")
    return dk, dv


class Infeasible(Exception):
    """No partition fits the budget (some sequence is too large even with full recompute)."""


def plan_bruteforce(lengths, budget: int, n_heads=16, head_dim=128, elt_bytes=2, n_layers=1,
                    const_bytes=0, fixed_cost=1 << 24, fwd_time=None):
    """Best plan by enumeration of all 2^(n-1) contiguous splits of the length-sorted list.
    fwd_time (optional, one integer per sequence) replaces the 2 L^2 forward-time model (Section 3.5).
    Returns (mb_id list[n], recompute list[K], cost int)."""
    lengths = np.ascontiguousarray(lengths, dtype=np.int32)
    n = int(lengths.size)
    wt = None if fwd_time is None else np.ascontiguousarray(fwd_time, dtype=np.int64)
    if wt is not None and wt.size != n:
        raise ValueError("fwd_time needs one entry per sequence")
    params = PlanParams(n_heads, head_dim, elt_bytes, n_layers, const_bytes, fixed_cost)
    mb = np.zeros(max(n, 1), np.int32)
    rec = np.zeros(max(n, 1), np.int32)
    n_mb = ctypes.c_int32(0)
    lo, hi = ctypes.c_uint64(0), ctypes.c_uint64(0)
    rc = _load().oracle_plan_bruteforce_weighted(_p(lengths, ctypes.c_int32),
                                                 None if wt is None else _p(wt, ctypes.c_int64), n, int(budget),
                                                 ctypes.byref(params), _p(mb, ctypes.c_int32), ctypes.byref(n_mb),
                                                 _p(rec, ctypes.c_int32), ctypes.byref(lo), ctypes.byref(hi))
    if rc == 3:
        raise Infeasible()
    if rc:
        raise ValueError(f"oracle_plan_bruteforce rejected its arguments ({rc})")
    K = n_mb.value
    return mb[:n].tolist(), rec[:K].tolist(), (hi.value << 64) | lo.value


def inter_bruteforce(times, g_min: int = 1, g_max: int = 4):
    """Best accumulation-step vector by enumeration of every vector within the G_max bound.
    Returns (g list[n], idle int).  Raises ValueError when the search space exceeds 5e7 vectors."""
    t = np.ascontiguousarray(times, dtype=np.int64)
    n = int(t.size)
    g = np.zeros(max(n, 1), np.int32)
    lo, hi = ctypes.c_uint64(0), ctypes.c_uint64(0)
    rc = _load().oracle_inter_bruteforce(_p(t, ctypes.c_int64), n, int(g_min), int(g_max), _p(g, ctypes.c_int32),
                                         ctypes.byref(lo), ctypes.byref(hi))
    if rc:
        raise ValueError(f"oracle_inter_bruteforce rejected its arguments or the space is too large ({rc})")
    return g[:n].tolist(), (hi.value << 64) | lo.value


from .intra_oracle import intra_select  # noqa: E402,F401  (Algorithm 1, plain Python)
from . import profile_oracle, shard_oracle  # noqa: E402,F401
