"""Dual-layer profiling of the attention kernels on the current GPU (Section 3.5 of the paper).

The paper measures, for every candidate setting, two layers: the first only warms up, the second
gives the per-layer forward time t_f, backward time t_b and activation memory m, from which the
whole model is extrapolated as Lambda * (2 t_f + t_b) + T_C under full recomputation.  Here a
"layer" is the packed attention forward + backward of this library and the candidates are sequence
length buckets (sequence-parallel size is 1 on one GPU).  The table feeds dcp_plan_profiled, which
replaces the planner's L^2 stand-in for t_f by these measurements.

Only host logic lives here: which buckets to run and what to keep.  The timed work is the library's
kernels, timed by the library's own CUDA events; interpolation between buckets (dcp_profile_interp),
the modelled time of a micro-batch (dcp_model_time, Eq. 4-5) and the candidate rows of Algorithm 1
(dcp_intra_candidate_from_profile) are computed by the library.
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import Callable, List, Optional, Sequence, Tuple


@dataclass
class ProfileTable:
    """Per-sequence, per-layer times in integer nanoseconds at ascending bucket lengths."""
    lengths: List[int]
    t_f_ns: List[int]
    t_b_ns: List[int]
    m_bytes: List[int]          # what a layer that is not recomputed keeps: q, k, v, o

    def __post_init__(self):
        n = len(self.lengths)
        if n < 1 or not (len(self.t_f_ns) == len(self.t_b_ns) == len(self.m_bytes) == n):
            raise ValueError("a profile needs at least one bucket and equally long columns")
        if any(b <= a for a, b in zip(self.lengths, self.lengths[1:])) or self.lengths[0] < 1:
            raise ValueError("bucket lengths must be positive and strictly ascending")
        if any(t < 0 for t in self.t_f_ns + self.t_b_ns):
            raise ValueError("negative time in profile")

    def fwd_times(self, lengths: Sequence[int]) -> List[int]:
        from . import binding
        return binding.dcp_profile_interp(self.lengths, self.t_f_ns, lengths)

    def bwd_times(self, lengths: Sequence[int]) -> List[int]:
        from . import binding
        return binding.dcp_profile_interp(self.lengths, self.t_b_ns, lengths)

    def fwd_time(self, L: int) -> int:
        return self.fwd_times([L])[0]

    def bwd_time(self, L: int) -> int:
        return self.bwd_times([L])[0]

    def model_time(self, lengths: Sequence[int], n_layers: int, recompute: int, fixed_cost_ns: int = 0) -> int:
        """Eq. 4-5: T = Lambda (t_f + t_b) + r t_f + T_C for one micro-batch."""
        from . import binding
        return binding.dcp_model_time(self.fwd_times(lengths), self.bwd_times(lengths), n_layers, recompute,
                                      fixed_cost_ns)


def _gpu_layer(n_heads: int, head_dim: int, causal: bool, device) -> Callable[[List[int]], Tuple[float, float]]:
    """One 'layer' = forward + backward over a packed batch; returns (forward ms, backward ms)
    from the library's per-kernel CUDA-event timers."""
    import torch
    from . import binding, inputs

    def run(lengths: List[int]) -> Tuple[float, float]:
        T = sum(lengths)
        q, k, v, g = inputs.make_qkvg_device(T, n_heads, head_dim, 77, device)
        cu = torch.tensor([0] + list(torch.tensor(lengths).cumsum(0).tolist()), dtype=torch.int32, device=device)
        ws = binding.alloc_workspace(T, len(lengths), n_heads, head_dim, True, device)
        binding.dcp_profile_enable(True)
        binding.dcp_profile_read()
        o, lse = binding.dcp_varlen_attn_fwd(q, k, v, cu, max(lengths), causal, workspace=ws)
        torch.cuda.synchronize()
        f = binding.dcp_profile_read()
        binding.dcp_varlen_attn_bwd(q, k, v, o, g, lse, cu, max(lengths), causal, workspace=ws)
        torch.cuda.synchronize()
        b = binding.dcp_profile_read()
        binding.dcp_profile_enable(False)
        binding.dcp_query_status(ws)
        return sum(ms for ms, _ in f.values()), sum(ms for ms, _ in b.values())

    return run


def dual_layer_profile(bucket_lengths: Sequence[int], n_heads: int, head_dim: int, causal: bool, device="cuda",
                       fill_tokens: int = 1 << 16, elt_bytes: int = 2,
                       run_layer: Optional[Callable[[List[int]], Tuple[float, float]]] = None) -> ProfileTable:
    """Measure every bucket twice and keep the second run (the first layer only warms up).

    A bucket is run as a batch of equal sequences holding about `fill_tokens` tokens, so that the
    GPU is full as it is inside a real batch, and the batch time is divided by the number of copies.
    `run_layer(lengths) -> (forward ms, backward ms)` defaults to this library's kernels on `device`.
    """
    buckets = sorted(set(int(L) for L in bucket_lengths))
    if not buckets or buckets[0] < 1:
        raise ValueError("bucket lengths must be positive")
    run = run_layer if run_layer is not None else _gpu_layer(n_heads, head_dim, causal, device)
    t_f, t_b, m = [], [], []
    for L in buckets:
        copies = max(1, -(-fill_tokens // L))
        run([L] * copies)                                   # first layer: warm-up, discarded
        f_ms, b_ms = run([L] * copies)                      # second layer: recorded
        from . import binding
        t_f.append(int(round(f_ms * 1e6)) // copies)
        t_b.append(int(round(b_ms * 1e6)) // copies)
        m.append(binding.dcp_activation_bytes(L, n_heads, head_dim, elt_bytes)[0])
    return ProfileTable(buckets, t_f, t_b, m)


def _gpu_layer_head_group(n_heads: int, sp_size: int, head_dim: int, causal: bool, device) -> Callable[[List[int]], Tuple[float, float]]:
    """One rank's share of a 'layer' under head-sharded sequence parallelism of size sp_size: forward + backward
    on the first n_heads / sp_size heads, in place inside full-width [T, n_heads, head_dim] tensors (the strided
    entry points, as a rank of a group runs them).  Returns (forward ms, backward ms)."""
    import torch
    from . import binding, inputs

    def run(lengths: List[int]) -> Tuple[float, float]:
        T, hg = sum(lengths), n_heads // sp_size
        q, k, v, g = inputs.make_qkvg_device(T, n_heads, head_dim, 77, device)
        o, dq, dk, dv = (torch.empty_like(q) for _ in range(4))
        cu = torch.tensor([0] + list(torch.tensor(lengths).cumsum(0).tolist()), dtype=torch.int32, device=device)
        hs = slice(0, hg)
        binding.dcp_profile_enable(True)
        binding.dcp_profile_read()
        _, lse = binding.dcp_varlen_attn_fwd_strided(q[:, hs], k[:, hs], v[:, hs], cu, max(lengths), causal, o[:, hs])
        torch.cuda.synchronize()
        f = binding.dcp_profile_read()
        binding.dcp_varlen_attn_bwd_strided(q[:, hs], k[:, hs], v[:, hs], o[:, hs], g[:, hs], lse, cu, max(lengths), causal,
                                            dq[:, hs], dk[:, hs], dv[:, hs])
        torch.cuda.synchronize()
        b = binding.dcp_profile_read()
        binding.dcp_profile_enable(False)
        return sum(ms for ms, _ in f.values()), sum(ms for ms, _ in b.values())

    return run


def intra_candidates(seq_len: int, batch_sizes: Sequence[int], n_heads: int, head_dim: int, causal: bool, n_layers: int,
                     device="cuda", elt_bytes: int = 2, const_bytes: int = 0, fixed_cost_ns: int = 0,
                     run_layer: Optional[Callable[[List[int]], Tuple[float, float]]] = None,
                     sp_sizes: Sequence[int] = (1,)):
    """The candidate table Algorithm 1 takes, for sequences of one length: one row (b, p) per batch size b and
    sequence-parallel size p, measured the dual-layer way (the batch of b sequences runs twice, the second run
    is kept).  Row = (b, p, t_f, m, T_(b,p), M_(b,p)) with t_f the measured forward time of one layer for the
    whole batch in ns, m the bytes a layer keeps when it is not recomputed, T = Lambda (2 t_f + t_b) + T_C the
    modelled time with every layer recomputed (Section 3.5) and M = Lambda m_inp + M_C (Eq. 6 at r = Lambda).
    For p > 1 a row describes ONE RANK of a head-sharded group (Section 4.1): its time is that of its
    n_heads / p heads over all tokens, measured on this GPU through the strided entry points, and its memory
    that of its 1 / p of the tokens.  What a row for p > 1 leaves out is the time the tiles take to cross
    NVLink, which one GPU cannot show: the ranks of a group fetch remote tiles inside the same kernels."""
    from . import binding
    rows = []
    for p in sp_sizes:
        if p < 1 or n_heads % p != 0:
            raise ValueError(f"sequence-parallel size {p} does not divide {n_heads} heads")
        if run_layer is not None:
            run = run_layer
        elif p == 1:
            run = _gpu_layer(n_heads, head_dim, causal, device)
        else:
            run = _gpu_layer_head_group(n_heads, p, head_dim, causal, device)
        for b in batch_sizes:
            run([seq_len] * b)                                  # first layer: warm-up, discarded
            f_ms, b_ms = run([seq_len] * b)                     # second layer: recorded
            act, inp = binding.dcp_activation_bytes(-(-b * seq_len // p), n_heads, head_dim, elt_bytes)
            rows.append(binding.dcp_intra_candidate_from_profile(b, p, int(round(f_ms * 1e6)), int(round(b_ms * 1e6)), act, inp,
                                                                 n_layers, const_bytes, fixed_cost_ns))
    return rows


def select_group_setting(candidates, mem_capacity: int, n_layers: int) -> Tuple[int, int, int]:
    """(batch size, recompute count, modelled time) Algorithm 1 picks from a candidate table."""
    from . import binding
    idx, r, t = binding.dcp_intra_select(candidates, mem_capacity, n_layers)
    return candidates[idx][0], r, t
