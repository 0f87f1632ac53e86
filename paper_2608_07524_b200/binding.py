"""ctypes binding over libdcp.so: the same entry points as include/dcp.h, with torch tensors
marshalled to raw pointers.  No step of the computation runs here; if the library is missing the
calls raise instead of falling back to anything else.
"""
from __future__ import annotations

import ctypes
import os
import threading
from typing import List, Optional, Tuple

_DIR = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_DIR, "libdcp.so")

DCP_OK, DCP_ERR_INVALID_ARG, DCP_ERR_INFEASIBLE, DCP_ERR_UNSUPPORTED = 0, 1, 2, 3
DCP_ERR_WORKSPACE, DCP_ERR_CUDA, DCP_ERR_TIMEOUT, DCP_ERR_OVERFLOW = 4, 5, 6, 7

_lock = threading.Lock()
_lib = None


class DcpError(RuntimeError):
    def __init__(self, code: int, message: str):
        super().__init__(f"libdcp error {code}: {message}")
        self.code = code


class PlanParams(ctypes.Structure):
    _fields_ = [("n_heads", ctypes.c_int32), ("head_dim", ctypes.c_int32),
                ("elt_bytes", ctypes.c_int32), ("n_layers", ctypes.c_int32),
                ("const_bytes", ctypes.c_int64), ("fixed_cost", ctypes.c_int64)]


class IntraCandidate(ctypes.Structure):
    _fields_ = [("batch_size", ctypes.c_int32), ("sp_size", ctypes.c_int32), ("t_f", ctypes.c_int64),
                ("m", ctypes.c_int64), ("time_full", ctypes.c_int64), ("mem_full", ctypes.c_int64)]


def lib():
    """The loaded library.  Raises if libdcp.so has not been built (python -m paper_2608_07524_b200.build)."""
    global _lib
    with _lock:
        if _lib is None:
            if not os.path.exists(LIB_PATH):
                raise FileNotFoundError(
                    f"{LIB_PATH} is missing: build it with `python -m paper_2608_07524_b200.build`; "
                    "there is no fallback path")
            L = ctypes.CDLL(LIB_PATH)
            i32, i64, vp, f32 = ctypes.c_int32, ctypes.c_int64, ctypes.c_void_p, ctypes.c_float
            i32p = ctypes.POINTER(ctypes.c_int32)
            szp = ctypes.POINTER(ctypes.c_size_t)
            i64p = ctypes.POINTER(ctypes.c_int64)
            L.dcp_plan.argtypes = [i32p, i32, i64, ctypes.POINTER(PlanParams), i32p, i32p, i32p,
                                   ctypes.POINTER(ctypes.c_int64)]
            L.dcp_plan.restype = ctypes.c_int
            L.dcp_plan_profiled.argtypes = [i32p, i64p, i32, i64, ctypes.POINTER(PlanParams), i32p, i32p, i32p,
                                            ctypes.POINTER(ctypes.c_int64)]
            L.dcp_plan_profiled.restype = ctypes.c_int
            L.dcp_inter_plan.argtypes = [i64p, i32, i32, i32, i32p, i64p, i64p]
            L.dcp_intra_select.argtypes = [ctypes.POINTER(IntraCandidate), i32, i64, i32, i32p, i32p, i64p]
            L.dcp_intra_select.restype = ctypes.c_int
            L.dcp_inter_plan.restype = ctypes.c_int
            L.dcp_varlen_attn_workspace.argtypes = [i32, i32, i32, i32, szp, szp]
            L.dcp_varlen_attn_workspace.restype = ctypes.c_int
            L.dcp_varlen_attn_fwd.argtypes = [vp, vp, vp, vp, i32, i32, i32, i32, i32, i32, f32, vp, vp, vp,
                                              ctypes.c_size_t, vp]
            L.dcp_varlen_attn_fwd.restype = ctypes.c_int
            L.dcp_varlen_attn_bwd.argtypes = [vp, vp, vp, vp, vp, vp, vp, i32, i32, i32, i32, i32, i32, f32,
                                              vp, vp, vp, vp, ctypes.c_size_t, vp]
            L.dcp_varlen_attn_bwd.restype = ctypes.c_int
            L.dcp_varlen_attn_fwd_noalloc.argtypes = [vp, vp, vp, vp, i32, i32, i32, i32, i32, i32, f32, vp, vp, vp]
            L.dcp_varlen_attn_fwd_noalloc.restype = ctypes.c_int
            L.dcp_query_status.argtypes = [vp, vp]
            L.dcp_query_status.restype = ctypes.c_int
            L.dcp_profile_enable.argtypes = [ctypes.c_int]
            L.dcp_profile_enable.restype = ctypes.c_int
            L.dcp_profile_read.argtypes = [ctypes.POINTER(ctypes.c_float), ctypes.POINTER(ctypes.c_int64)]
            L.dcp_profile_read.restype = ctypes.c_int
            L.dcp_launch_count.argtypes = []
            L.dcp_launch_count.restype = ctypes.c_int64
            L.dcp_last_error.argtypes = []
            L.dcp_last_error.restype = ctypes.c_char_p
            _lib = L
    return _lib


def _check(rc: int):
    if rc != DCP_OK:
        raise DcpError(rc, lib().dcp_last_error().decode(errors="replace"))


KERNEL_NAMES = ("prep", "fwd", "bwd_pre", "bwd_main", "bwd_post")


def dcp_profile_enable(on: bool) -> None:
    _check(lib().dcp_profile_enable(int(bool(on))))


def dcp_profile_read():
    """{kernel name: (device ms, launches)} accumulated since the previous read."""
    ms = (ctypes.c_float * len(KERNEL_NAMES))()
    n = (ctypes.c_int64 * len(KERNEL_NAMES))()
    _check(lib().dcp_profile_read(ms, n))
    return {name: (float(ms[i]), int(n[i])) for i, name in enumerate(KERNEL_NAMES)}


def dcp_launch_count() -> int:
    return int(lib().dcp_launch_count())


def dcp_plan(lengths, hbm_budget_bytes: int, n_heads: int = 16, head_dim: int = 128, elt_bytes: int = 2,
             n_layers: int = 1, const_bytes: int = 0, fixed_cost: int = 1 << 24
             ) -> Tuple[List[int], List[int], int]:
    """(mb_id [n], recompute [K], cost) for one batch of sequence lengths under an HBM budget."""
    n = len(lengths)
    arr = (ctypes.c_int32 * max(n, 1))(*[int(x) for x in lengths])
    mb = (ctypes.c_int32 * max(n, 1))()
    rec = (ctypes.c_int32 * max(n, 1))()
    n_mb = ctypes.c_int32(0)
    cost = ctypes.c_int64(0)
    params = PlanParams(n_heads, head_dim, elt_bytes, n_layers, const_bytes, fixed_cost)
    _check(lib().dcp_plan(arr, n, int(hbm_budget_bytes), ctypes.byref(params), mb, ctypes.byref(n_mb), rec,
                          ctypes.byref(cost)))
    return list(mb[:n]), list(rec[:n_mb.value]), int(cost.value)


def dcp_plan_profiled(lengths, fwd_time, hbm_budget_bytes: int, n_heads: int = 16, head_dim: int = 128,
                      elt_bytes: int = 2, n_layers: int = 1, const_bytes: int = 0, fixed_cost: int = 0
                      ) -> Tuple[List[int], List[int], int]:
    """dcp_plan with a profiled per-layer forward time per sequence (Section 3.5) instead of the L^2 model;
    fixed_cost is in the unit of fwd_time."""
    n = len(lengths)
    if len(fwd_time) != n:
        raise ValueError("fwd_time needs one entry per sequence")
    arr = (ctypes.c_int32 * max(n, 1))(*[int(x) for x in lengths])
    wt = (ctypes.c_int64 * max(n, 1))(*[int(x) for x in fwd_time])
    mb = (ctypes.c_int32 * max(n, 1))()
    rec = (ctypes.c_int32 * max(n, 1))()
    n_mb = ctypes.c_int32(0)
    cost = ctypes.c_int64(0)
    params = PlanParams(n_heads, head_dim, elt_bytes, n_layers, const_bytes, fixed_cost)
    _check(lib().dcp_plan_profiled(arr, wt, n, int(hbm_budget_bytes), ctypes.byref(params), mb, ctypes.byref(n_mb),
                                   rec, ctypes.byref(cost)))
    return list(mb[:n]), list(rec[:n_mb.value]), int(cost.value)


def dcp_inter_plan(times, g_min: int = 1, g_max: int = 4) -> Tuple[List[int], int, int]:
    """(g [n], idle, iteration_time): accumulation steps balancing n side-by-side batches (Eq. 3)."""
    n = len(times)
    arr = (ctypes.c_int64 * max(n, 1))(*[int(x) for x in times])
    g = (ctypes.c_int32 * max(n, 1))()
    idle, it = ctypes.c_int64(0), ctypes.c_int64(0)
    _check(lib().dcp_inter_plan(arr, n, int(g_min), int(g_max), g, ctypes.byref(idle), ctypes.byref(it)))
    return list(g[:n]), int(idle.value), int(it.value)


def dcp_intra_select(candidates, mem_capacity: int, n_layers: int) -> Tuple[int, int, int]:
    """(index, recompute, time) of the throughput-optimal candidate (Algorithm 1).  Each candidate is
    (batch_size, sp_size, t_f, m, time_full, mem_full), profiled with every layer recomputed."""
    n = len(candidates)
    arr = (IntraCandidate * max(n, 1))(*[IntraCandidate(*[int(x) for x in c]) for c in candidates])
    best, rec, t = ctypes.c_int32(0), ctypes.c_int32(0), ctypes.c_int64(0)
    _check(lib().dcp_intra_select(arr, n, int(mem_capacity), int(n_layers), ctypes.byref(best), ctypes.byref(rec),
                                  ctypes.byref(t)))
    return int(best.value), int(rec.value), int(t.value)


def dcp_varlen_attn_workspace(total_tokens: int, n_seqs: int, n_heads: int, head_dim: int) -> Tuple[int, int]:
    fwd, bwd = ctypes.c_size_t(0), ctypes.c_size_t(0)
    _check(lib().dcp_varlen_attn_workspace(total_tokens, n_seqs, n_heads, head_dim, ctypes.byref(fwd),
                                           ctypes.byref(bwd)))
    return int(fwd.value), int(bwd.value)


def _ptr(t) -> Optional[int]:
    return None if t is None else t.data_ptr()


def _stream(stream) -> Optional[int]:
    import torch
    s = torch.cuda.current_stream() if stream is None else stream
    return s.cuda_stream or None


def _require(t, dtype, name):
    if not t.is_cuda or not t.is_contiguous() or t.dtype != dtype:
        raise TypeError(f"{name} must be a contiguous CUDA tensor of dtype {dtype}")


def alloc_workspace(total_tokens: int, n_seqs: int, n_heads: int, head_dim: int, backward: bool, device):
    """A uint8 tensor large enough for the forward (or backward) call; torch's allocator returns
    512-byte aligned blocks."""
    import torch
    fwd, bwd = dcp_varlen_attn_workspace(total_tokens, n_seqs, n_heads, head_dim)
    return torch.empty(bwd if backward else fwd, dtype=torch.uint8, device=device)


def dcp_varlen_attn_fwd(q, k, v, cu_seqlens, max_seqlen: int, causal: bool, softmax_scale: float = 0.0,
                        out=None, lse=None, workspace=None, stream=None):
    """o [T,H,d] bf16 and lse [H,T] fp32.  cu_seqlens: int32 CUDA tensor [B+1].  Enqueues only."""
    import torch
    for name, t in (("q", q), ("k", k), ("v", v)):
        _require(t, torch.bfloat16, name)
    _require(cu_seqlens, torch.int32, "cu_seqlens")
    T, H, d = q.shape
    n_seqs = cu_seqlens.numel() - 1
    o = torch.empty_like(q) if out is None else out
    lse = torch.empty((H, T), dtype=torch.float32, device=q.device) if lse is None else lse
    ws = alloc_workspace(T, n_seqs, H, d, False, q.device) if workspace is None else workspace
    _check(lib().dcp_varlen_attn_fwd(_ptr(q), _ptr(k), _ptr(v), _ptr(cu_seqlens), n_seqs, T, int(max_seqlen), H, d,
                                     int(bool(causal)), float(softmax_scale), _ptr(o), _ptr(lse), _ptr(ws),
                                     ws.numel(), _stream(stream)))
    return o, lse


NOALLOC_MAX_SEQS = 4096


def dcp_varlen_attn_fwd_noalloc(q, k, v, cu_seqlens, max_seqlen: int, causal: bool, out, lse,
                                softmax_scale: float = 0.0, stream=None):
    """Forward attention for callers that cannot allocate device memory: the caller supplies `out`
    [T,H,d] bf16 and `lse` [H,T] fp32; the work-list scratch is a fixed array inside the library (at
    most NOALLOC_MAX_SEQS sequences).  This wrapper allocates nothing either.  Calls on one device
    share that array, so do not let two of them overlap on the GPU."""
    import torch
    for name, t in (("q", q), ("k", k), ("v", v), ("out", out)):
        _require(t, torch.bfloat16, name)
    _require(lse, torch.float32, "lse")
    _require(cu_seqlens, torch.int32, "cu_seqlens")
    T, H, d = q.shape
    _check(lib().dcp_varlen_attn_fwd_noalloc(_ptr(q), _ptr(k), _ptr(v), _ptr(cu_seqlens), cu_seqlens.numel() - 1, T,
                                             int(max_seqlen), H, d, int(bool(causal)), float(softmax_scale),
                                             _ptr(out), _ptr(lse), _stream(stream)))
    return out, lse


def dcp_varlen_attn_bwd(q, k, v, o, d_o, lse, cu_seqlens, max_seqlen: int, causal: bool,
                        softmax_scale: float = 0.0, dq=None, dk=None, dv=None, workspace=None, stream=None):
    """dq, dk, dv [T,H,d] bf16 for the loss sum(o * d_o).  Enqueues only."""
    import torch
    for name, t in (("q", q), ("k", k), ("v", v), ("o", o), ("d_o", d_o)):
        _require(t, torch.bfloat16, name)
    _require(lse, torch.float32, "lse")
    _require(cu_seqlens, torch.int32, "cu_seqlens")
    T, H, d = q.shape
    n_seqs = cu_seqlens.numel() - 1
    dq = torch.empty_like(q) if dq is None else dq
    dk = torch.empty_like(q) if dk is None else dk
    dv = torch.empty_like(q) if dv is None else dv
    ws = alloc_workspace(T, n_seqs, H, d, True, q.device) if workspace is None else workspace
    _check(lib().dcp_varlen_attn_bwd(_ptr(q), _ptr(k), _ptr(v), _ptr(o), _ptr(d_o), _ptr(lse), _ptr(cu_seqlens),
                                     n_seqs, T, int(max_seqlen), H, d, int(bool(causal)), float(softmax_scale),
                                     _ptr(dq), _ptr(dk), _ptr(dv), _ptr(ws), ws.numel(), _stream(stream)))
    return dq, dk, dv


def dcp_query_status(workspace, stream=None) -> None:
    """Synchronises the stream and raises DcpError if a kernel reported a failure."""
    _check(lib().dcp_query_status(_ptr(workspace), _stream(stream)))
