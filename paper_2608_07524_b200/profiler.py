"""Dual-layer profiling of the attention kernels on the current GPU (Section 3.5 of the paper).

The paper measures, for every candidate setting, two layers: the first only warms up, the second
gives the per-layer forward time t_f, backward time t_b and activation memory m, from which the
whole model is extrapolated as Lambda * (2 t_f + t_b) + T_C under full recomputation.  Here a
"layer" is the packed attention forward + backward of this library and the candidates are sequence
length buckets (sequence-parallel size is 1 on one GPU).  The table feeds dcp_plan_profiled, which
replaces the planner's L^2 stand-in for t_f by these measurements.

Only host logic lives here: which buckets to run, what to keep, and integer interpolation between
buckets.  The timed work is the library's kernels, timed by the library's own CUDA events.
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

    def _interp(self, col: Sequence[int], L: int) -> int:
        """Integer interpolation, floor division throughout:
        below the first bucket linear in L (short sequences are bound by memory traffic, which is
        linear in tokens); between buckets linear; above the last bucket quadratic in L."""
        if L < 1:
            raise ValueError("length must be >= 1")
        xs = self.lengths
        if L <= xs[0]:
            return col[0] * L // xs[0]
        if L >= xs[-1]:
            return col[-1] * L * L // (xs[-1] * xs[-1])
        hi = next(i for i, x in enumerate(xs) if x >= L)
        lo = hi - 1
        return col[lo] + (col[hi] - col[lo]) * (L - xs[lo]) // (xs[hi] - xs[lo])

    def fwd_time(self, L: int) -> int:
        return self._interp(self.t_f_ns, L)

    def bwd_time(self, L: int) -> int:
        return self._interp(self.t_b_ns, L)

    def model_time(self, lengths: Sequence[int], n_layers: int, recompute: int, fixed_cost_ns: int = 0) -> int:
        """Eq. 4-5: T = Lambda (t_f + t_b) + r t_f + T_C for one micro-batch."""
        tf = sum(self.fwd_time(L) for L in lengths)
        tb = sum(self.bwd_time(L) for L in lengths)
        return n_layers * (tf + tb) + recompute * tf + fixed_cost_ns


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
        t_f.append(int(round(f_ms * 1e6)) // copies)
        t_b.append(int(round(b_ms * 1e6)) // copies)
        m.append(4 * L * n_heads * head_dim * elt_bytes)
    return ProfileTable(buckets, t_f, t_b, m)
