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
            L.dcp_varlen_attn_fwd_strided.argtypes = [vp, vp, vp, vp, i32, i32, i32, i32, i32, i64, i32, f32, vp, vp, vp,
                                                      ctypes.c_size_t, vp]
            L.dcp_varlen_attn_fwd_strided.restype = ctypes.c_int
            L.dcp_varlen_attn_bwd_strided.argtypes = [vp, vp, vp, vp, vp, vp, vp, i32, i32, i32, i32, i32, i64, i32, f32,
                                                      vp, vp, vp, vp, ctypes.c_size_t, vp]
            L.dcp_varlen_attn_bwd_strided.restype = ctypes.c_int
            L.dcp_varlen_attn_fwd_noalloc.argtypes = [vp, vp, vp, vp, i32, i32, i32, i32, i32, i32, f32, vp, vp, vp]
            L.dcp_varlen_attn_fwd_noalloc.restype = ctypes.c_int
            L.dcp_query_status.argtypes = [vp, vp]
            L.dcp_query_status.restype = ctypes.c_int
            L.dcp_noalloc_status.argtypes = [vp]
            L.dcp_noalloc_status.restype = ctypes.c_int
            L.dcp_selftest_wait_timeout.argtypes = [vp, ctypes.c_uint32, vp]
            L.dcp_selftest_wait_timeout.restype = ctypes.c_int
            L.dcp_set_work_order.argtypes = [ctypes.c_int]
            L.dcp_set_work_order.restype = ctypes.c_int
            L.dcp_set_short_sequence_path.argtypes = [ctypes.c_int]
            L.dcp_set_short_sequence_path.restype = ctypes.c_int
            L.dcp_read_cta_spans.argtypes = [vp, i32, vp, i64p, i64p, i32p]
            L.dcp_read_cta_spans.restype = ctypes.c_int
            L.dcp_plan_segments.argtypes = [i32p, i32p, i32, i32, i32, i32p, i32p, i32p, i32p, i32p, i32, i32p]
            L.dcp_plan_segments.restype = ctypes.c_int
            L.dcp_copy_segments.argtypes = [vp, vp, vp, i32, i64, i32, i64, i64, i32, vp]
            L.dcp_copy_segments.restype = ctypes.c_int
            L.dcp_profile_interp.argtypes = [i32p, i64p, i32, i32p, i32, i64p]
            L.dcp_profile_interp.restype = ctypes.c_int
            L.dcp_model_time.argtypes = [i64p, i64p, i32, i32, i32, i64, i64p]
            L.dcp_model_time.restype = ctypes.c_int
            L.dcp_intra_candidate_from_profile.argtypes = [i32, i32, i64, i64, i64, i64, i32, i64, i64,
                                                           ctypes.POINTER(IntraCandidate)]
            L.dcp_intra_candidate_from_profile.restype = ctypes.c_int
            L.dcp_activation_bytes.argtypes = [i64, i32, i32, i32, i64p, i64p]
            L.dcp_activation_bytes.restype = ctypes.c_int
            L.dcp_length_group_plan.argtypes = [i32, i32, i32p, i32p]
            L.dcp_length_group_plan.restype = ctypes.c_int
            L.dcp_shard_sequences.argtypes = [i32p, i32, i32, i32p, i64p]
            L.dcp_shard_sequences.restype = ctypes.c_int
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


def _require_head_group(t, name, stride=None):
    """A bf16 CUDA view [T, Hg, d] of a group of heads inside a wider [T, H, d] tensor: unit stride along
    d, heads d apart, tokens `stride` apart.  Returns the token stride."""
    import torch
    if not t.is_cuda or t.dtype != torch.bfloat16 or t.dim() != 3:
        raise TypeError(f"{name} must be a bf16 CUDA tensor [T, heads, head_dim]")
    T, Hg, d = t.shape
    st = t.stride()
    if st[2] != 1 or (Hg > 1 and st[1] != d) or (T > 1 and st[0] < Hg * d) or (stride is not None and T > 1 and st[0] != stride):
        raise TypeError(f"{name} must be a group of adjacent heads of a [T, H, d] tensor (same token stride for all tensors)")
    return int(st[0]) if T > 1 else (stride if stride is not None else Hg * d)


def dcp_varlen_attn_fwd_strided(q, k, v, cu_seqlens, max_seqlen: int, causal: bool, out, softmax_scale: float = 0.0,
                                lse=None, workspace=None, stream=None):
    """Forward attention on a group of heads inside wider tensors (views such as x[:, h0:h1, :]); `out` is a
    view of the same kind.  lse [Hg, T] fp32 is contiguous and belongs to the group.  Enqueues only."""
    import torch
    stride = _require_head_group(q, "q")
    for name, t in (("k", k), ("v", v), ("out", out)):
        _require_head_group(t, name, stride)
    _require(cu_seqlens, torch.int32, "cu_seqlens")
    T, Hg, d = q.shape
    n_seqs = cu_seqlens.numel() - 1
    lse = torch.empty((Hg, T), dtype=torch.float32, device=q.device) if lse is None else lse
    ws = alloc_workspace(T, n_seqs, Hg, d, False, q.device) if workspace is None else workspace
    _check(lib().dcp_varlen_attn_fwd_strided(_ptr(q), _ptr(k), _ptr(v), _ptr(cu_seqlens), n_seqs, T, int(max_seqlen), Hg,
                                             d, stride, int(bool(causal)), float(softmax_scale), _ptr(out), _ptr(lse),
                                             _ptr(ws), ws.numel(), _stream(stream)))
    return out, lse


def dcp_varlen_attn_bwd_strided(q, k, v, o, d_o, lse, cu_seqlens, max_seqlen: int, causal: bool, dq, dk, dv,
                                softmax_scale: float = 0.0, workspace=None, stream=None):
    """Backward attention on a group of heads inside wider tensors; dq, dk, dv are views of the same kind."""
    import torch
    stride = _require_head_group(q, "q")
    for name, t in (("k", k), ("v", v), ("o", o), ("d_o", d_o), ("dq", dq), ("dk", dk), ("dv", dv)):
        _require_head_group(t, name, stride)
    _require(lse, torch.float32, "lse")
    _require(cu_seqlens, torch.int32, "cu_seqlens")
    T, Hg, d = q.shape
    n_seqs = cu_seqlens.numel() - 1
    ws = alloc_workspace(T, n_seqs, Hg, d, True, q.device) if workspace is None else workspace
    _check(lib().dcp_varlen_attn_bwd_strided(_ptr(q), _ptr(k), _ptr(v), _ptr(o), _ptr(d_o), _ptr(lse), _ptr(cu_seqlens),
                                             n_seqs, T, int(max_seqlen), Hg, d, stride, int(bool(causal)),
                                             float(softmax_scale), _ptr(dq), _ptr(dk), _ptr(dv), _ptr(ws), ws.numel(),
                                             _stream(stream)))
    return dq, dk, dv


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
    """Synchronises the stream and raises DcpError if any call on this workspace since the previous
    query reported a failure (the device status word is sticky; the query clears it)."""
    _check(lib().dcp_query_status(_ptr(workspace), _stream(stream)))


def dcp_noalloc_status(stream=None) -> None:
    """dcp_query_status for the built-in scratch of dcp_varlen_attn_fwd_noalloc on the current device."""
    _check(lib().dcp_noalloc_status(_stream(stream)))


def dcp_selftest_wait_timeout(workspace, spin_limit: int = 1 << 10, stream=None) -> None:
    """Enqueues the self-test CTA whose bounded wait expires; dcp_query_status then raises DCP_ERR_TIMEOUT."""
    _check(lib().dcp_selftest_wait_timeout(_ptr(workspace), int(spin_limit), _stream(stream)))


def dcp_set_work_order(input_order: bool) -> None:
    """Measurement aid: list sequences as they come (True) instead of longest first (False, default)."""
    _check(lib().dcp_set_work_order(int(bool(input_order))))


def dcp_set_short_sequence_path(enabled: bool) -> None:
    """Measurement aid and test hook: batches whose declared max_seqlen is at most 32 run on the small per-sequence
    kernels (True, default) or on the tile kernels like every other batch (False)."""
    _check(lib().dcp_set_short_sequence_path(int(bool(enabled))))


def dcp_read_cta_spans(workspace, which: int, stream=None):
    """(begin_ns, end_ns) int64 numpy arrays, one entry per persistent CTA of the last forward (which = 0)
    or backward main (which = 1) launch on this workspace."""
    import numpy as np
    begin = np.zeros(256, np.int64)
    end = np.zeros(256, np.int64)
    n = ctypes.c_int32(0)
    i64p = ctypes.POINTER(ctypes.c_int64)
    _check(lib().dcp_read_cta_spans(_ptr(workspace), int(which), _stream(stream), begin.ctypes.data_as(i64p),
                                    end.ctypes.data_as(i64p), ctypes.byref(n)))
    return begin[: n.value].copy(), end[: n.value].copy()


def _i32(a):
    import numpy as np
    return np.ascontiguousarray(a, dtype=np.int32)


def _i32p(a):
    return a.ctypes.data_as(ctypes.POINTER(ctypes.c_int32))


def _i64p(a):
    return a.ctypes.data_as(ctypes.POINTER(ctypes.c_int64))


def dcp_plan_segments(lengths, mb_id, n_mb: int, max_rows: int = 64):
    """(mb_seq_offset [K+1], seq_index [n], mb_cu [n+K], seg_offset [K+1], seg [n_seg, 3]) as int32 numpy
    arrays: where each sequence of a planned batch lives in the batch and in its micro-batch."""
    import numpy as np
    lengths, mb_id = _i32(lengths), _i32(mb_id)
    n = int(lengths.size)
    cap = n + int(lengths.sum()) // int(max_rows)
    mb_seq_offset, seq_index = np.zeros(n_mb + 1, np.int32), np.zeros(max(n, 1), np.int32)
    mb_cu, seg_offset = np.zeros(n + n_mb, np.int32), np.zeros(n_mb + 1, np.int32)
    seg = np.zeros((max(cap, 1), 3), np.int32)
    n_seg = ctypes.c_int32(0)
    _check(lib().dcp_plan_segments(_i32p(lengths), _i32p(mb_id), n, int(n_mb), int(max_rows), _i32p(mb_seq_offset),
                                   _i32p(seq_index), _i32p(mb_cu), _i32p(seg_offset), _i32p(seg), cap,
                                   ctypes.byref(n_seg)))
    return mb_seq_offset, seq_index[:n], mb_cu, seg_offset, seg[: n_seg.value]


def dcp_copy_segments(src, dst, seg, n_seg: int, row_bytes: int, reverse: bool = False, n_planes: int = 1,
                      src_plane_bytes: int = 0, dst_plane_bytes: int = 0, stream=None) -> None:
    """Row-range copies between two CUDA tensors; seg is an int32 CUDA tensor [n_seg, 3].  Enqueues only."""
    _check(lib().dcp_copy_segments(_ptr(src), _ptr(dst), _ptr(seg), int(n_seg), int(row_bytes), int(n_planes),
                                   int(src_plane_bytes), int(dst_plane_bytes), int(bool(reverse)), _stream(stream)))


def dcp_profile_interp(bucket_len, bucket_val, lengths) -> List[int]:
    """Profiled per-sequence values at arbitrary lengths (Section 3.5; the rule is in include/dcp.h)."""
    import numpy as np
    xs, ys = _i32(bucket_len), np.ascontiguousarray(bucket_val, dtype=np.int64)
    ls = _i32(lengths)
    out = np.zeros(max(int(ls.size), 1), np.int64)
    _check(lib().dcp_profile_interp(_i32p(xs), _i64p(ys), int(xs.size), _i32p(ls), int(ls.size), _i64p(out)))
    return [int(x) for x in out[: ls.size]]


def dcp_model_time(fwd_time, bwd_time, n_layers: int, recompute: int, fixed_cost: int = 0) -> int:
    """Eq. 4-5 for one micro-batch: Lambda (sum t_f + sum t_b) + r sum t_f + T_C."""
    import numpy as np
    f, b = np.ascontiguousarray(fwd_time, dtype=np.int64), np.ascontiguousarray(bwd_time, dtype=np.int64)
    if f.size != b.size:
        raise ValueError("fwd_time and bwd_time need one entry per sequence each")
    t = ctypes.c_int64(0)
    _check(lib().dcp_model_time(_i64p(f), _i64p(b), int(f.size), int(n_layers), int(recompute), int(fixed_cost),
                                ctypes.byref(t)))
    return int(t.value)


def dcp_intra_candidate_from_profile(batch_size: int, sp_size: int, t_f: int, t_b: int, act_bytes: int, inp_bytes: int,
                                     n_layers: int, const_bytes: int = 0, fixed_cost: int = 0):
    """(b, p, t_f, m, T_(b,p), M_(b,p)): one row of Algorithm 1's candidate table from a dual-layer measurement."""
    c = IntraCandidate()
    _check(lib().dcp_intra_candidate_from_profile(int(batch_size), int(sp_size), int(t_f), int(t_b), int(act_bytes),
                                                  int(inp_bytes), int(n_layers), int(const_bytes), int(fixed_cost),
                                                  ctypes.byref(c)))
    return (c.batch_size, c.sp_size, c.t_f, c.m, c.time_full, c.mem_full)


def dcp_activation_bytes(tokens: int, n_heads: int, head_dim: int, elt_bytes: int = 2) -> Tuple[int, int]:
    """(m, m_inp) of the planner's memory model for `tokens` tokens: bytes a layer keeps when it is not
    recomputed, and the bytes of its input."""
    act, inp = ctypes.c_int64(0), ctypes.c_int64(0)
    _check(lib().dcp_activation_bytes(int(tokens), int(n_heads), int(head_dim), int(elt_bytes), ctypes.byref(act),
                                      ctypes.byref(inp)))
    return int(act.value), int(inp.value)


def dcp_length_group_plan(n_seqs: int, batch_size: int) -> Tuple[List[int], int]:
    """(mb_id [n_seqs], n_mb): consecutive sequences of a length group in micro-batches of batch_size."""
    mb = (ctypes.c_int32 * max(n_seqs, 1))()
    n_mb = ctypes.c_int32(0)
    _check(lib().dcp_length_group_plan(int(n_seqs), int(batch_size), mb, ctypes.byref(n_mb)))
    return list(mb[:n_seqs]), int(n_mb.value)


def dcp_shard_sequences(lengths, world_size: int):
    """(rank_of [n], load [world_size]): longest-first assignment of sequences to ranks by accumulated L^2."""
    import numpy as np
    ls = _i32(lengths)
    rank_of = np.zeros(max(int(ls.size), 1), np.int32)
    load = np.zeros(max(int(world_size), 1), np.int64)
    _check(lib().dcp_shard_sequences(_i32p(ls), int(ls.size), int(world_size), _i32p(rank_of), _i64p(load)))
    return [int(x) for x in rank_of[: ls.size]], [int(x) for x in load]
