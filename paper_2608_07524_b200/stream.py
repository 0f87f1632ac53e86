"""Host loop of the end-to-end stream: plan a batch, then run every micro-batch through the kernels.

Per batch (Section 3.1 of the paper: settings are re-chosen for every incoming batch and applied to
that batch's data):
    dcp_plan(lengths, budget)  ->  micro-batches (gradient-accumulation steps) and recompute counts
    dcp_plan_segments          ->  where each sequence sits in the batch and in its micro-batch
    for each micro-batch:      gather its sequences out of the batch (dcp_copy_segments); forward;
                               forward again if its recompute count > 0 (activation recomputation
                               re-runs the layer's forward before its backward, Section 3.4);
                               backward; scatter o, lse, dq, dk, dv back to the batch's order.
A plan with a single micro-batch runs in place, without copies.  All arithmetic happens in libdcp;
this module only owns buffers and issues calls.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import List, Optional, Sequence

import numpy as np

from . import binding

SEG_ROWS = 64      # rows per copy segment: 256 KB at 16 heads of 128, small enough for the copy grid to balance


@dataclass
class MicroBatch:
    lengths: Sequence[int]              # sequences the kernels see, in the order they are packed
    recompute: int                      # layers whose forward is re-run before backward
    seq_index: Optional[np.ndarray] = None   # input indices of the batch's sequences held here
    seg: Optional[np.ndarray] = None    # int32 [n_seg, 3] copy list (batch row, micro-batch row, rows); None = in place

    @property
    def total_tokens(self) -> int:
        return int(sum(self.lengths)) if isinstance(self.lengths, list) else int(np.asarray(self.lengths).sum())


@dataclass
class BatchPlan:
    mb_id: List[int]
    recompute: List[int]
    cost: int
    micro_batches: List[MicroBatch] = field(default_factory=list)


def plan_batch(lengths: Sequence[int], hbm_budget_bytes: int, n_heads: int, head_dim: int,
               n_layers: int = 1, fixed_cost: int = 1 << 24, profile=None) -> BatchPlan:
    """The plan of one batch and the layout of its micro-batches.  With `profile` (a
    profiler.ProfileTable) the per-layer forward time of every sequence comes from the measured table
    (Section 3.5) and fixed_cost is in nanoseconds; without it the planner uses its L^2 stand-in and
    fixed_cost is in its units.  Sequences keep their input order inside a micro-batch (the kernels
    order their own work); a single micro-batch is therefore the batch itself and needs no copy."""
    if profile is None:
        mb_id, recompute, cost = binding.dcp_plan(lengths, hbm_budget_bytes, n_heads=n_heads, head_dim=head_dim,
                                                  n_layers=n_layers, fixed_cost=fixed_cost)
    else:
        mb_id, recompute, cost = binding.dcp_plan_profiled(lengths, profile.fwd_times(lengths), hbm_budget_bytes,
                                                           n_heads=n_heads, head_dim=head_dim, n_layers=n_layers,
                                                           fixed_cost=fixed_cost)
    K = len(recompute)
    mb_seq_offset, seq_index, _, seg_offset, seg = binding.dcp_plan_segments(lengths, mb_id, K, SEG_ROWS)
    lens = np.asarray(lengths, dtype=np.int32)
    plan = BatchPlan(mb_id, recompute, cost)
    for k in range(K):
        idx = seq_index[mb_seq_offset[k]: mb_seq_offset[k + 1]]
        plan.micro_batches.append(MicroBatch(lens[idx], recompute[k], idx,
                                             None if K == 1 else seg[seg_offset[k]: seg_offset[k + 1]]))
    return plan


def plan_length_group(n_seqs: int, seq_len: int, batch_size: int, recompute: int) -> BatchPlan:
    """The plan of a group of n_seqs sequences of one length run with the setting Algorithm 1 selected
    for that length (Section 3.4): micro-batches of `batch_size` sequences each, every one with
    `recompute` recomputed layers.  Consecutive sequences share a micro-batch."""
    if recompute < 0:
        raise ValueError("need recompute >= 0")
    lengths = [int(seq_len)] * n_seqs
    mb_id, K = binding.dcp_length_group_plan(n_seqs, batch_size)
    mb_seq_offset, seq_index, _, seg_offset, seg = binding.dcp_plan_segments(lengths, mb_id, K, SEG_ROWS)
    lens = np.asarray(lengths, dtype=np.int32)
    plan = BatchPlan(mb_id, [int(recompute)] * K, 0)
    for k in range(K):
        idx = seq_index[mb_seq_offset[k]: mb_seq_offset[k + 1]]
        plan.micro_batches.append(MicroBatch(lens[idx], int(recompute), idx,
                                             None if K == 1 else seg[seg_offset[k]: seg_offset[k + 1]]))
    return plan


class _Buffers:
    """q, k, v, dO, o, dq, dk, dv [tokens, H, d] bf16 and lse [H * tokens] fp32 on the device."""

    def __init__(self, tokens, n_heads, head_dim, device, value_seed=None):
        import torch
        from . import inputs
        if value_seed is None:
            self.q, self.k, self.v, self.g = (torch.empty((tokens, n_heads, head_dim), dtype=torch.bfloat16, device=device)
                                              for _ in range(4))
        else:
            self.q, self.k, self.v, self.g = inputs.make_qkvg_device(tokens, n_heads, head_dim, value_seed, device)
        self.o, self.dq, self.dk, self.dv = (torch.empty_like(self.q) for _ in range(4))
        self.lse = torch.empty(n_heads * tokens, dtype=torch.float32, device=device)


class StreamRunner:
    """Runs planned batches out of pre-allocated device buffers.

    `batch` holds one batch in input order (inputs and results); micro-batches of a plan that splits
    the batch are gathered into `stage` (allocated on first need, sized like `batch`), run there and
    scattered back.  The synthetic stream reuses the first rows of `batch` for every batch (the values
    are random either way).
    """

    def __init__(self, max_tokens: int, max_seqs: int, n_heads: int, head_dim: int, causal: bool, device,
                 value_seed: int = 20):
        import torch
        self.torch = torch
        self.H, self.d, self.causal, self.device = n_heads, head_dim, causal, device
        self.max_tokens, self.max_seqs = max_tokens, max_seqs
        self.batch = _Buffers(max_tokens, n_heads, head_dim, device, value_seed)
        self.stage: Optional[_Buffers] = None
        # the single-batch benchmarks address the batch buffers directly
        self.q, self.k, self.v, self.g = self.batch.q, self.batch.k, self.batch.v, self.batch.g
        self.o, self.dq, self.dk, self.dv, self.lse = self.batch.o, self.batch.dq, self.batch.dk, self.batch.dv, self.batch.lse
        _, bwd_bytes = binding.dcp_varlen_attn_workspace(max_tokens, max_seqs, n_heads, head_dim)
        self.ws = torch.empty(bwd_bytes, dtype=torch.uint8, device=device)
        # cu_seqlens and copy lists travel through a small ring of pinned host / device slots; a slot is
        # reused only after the copy that read it has finished (tracked by an event per slot)
        self.n_slots = 16
        self.slot_ints = (max_seqs + 1) + 3 * (max_seqs + max_tokens // SEG_ROWS + 1)
        self.meta_host = torch.empty((self.n_slots, self.slot_ints), dtype=torch.int32).pin_memory()
        self.meta_host_np = self.meta_host.numpy()          # same memory: written with numpy
        self.meta_dev = torch.empty((self.n_slots, self.slot_ints), dtype=torch.int32, device=device)
        self.meta_events = [None] * self.n_slots
        self.calls = 0
        self.verify_recompute = False        # tests: compare the re-run forward with the first bit for bit
        self.recompute_mismatches = 0

    def _upload(self, lens: np.ndarray, seg: Optional[np.ndarray]):
        """cu_seqlens (and the copy list) of one micro-batch -> device, through the pinned ring."""
        torch = self.torch
        n = int(lens.size)
        slot = self.calls % self.n_slots
        self.calls += 1
        if self.meta_events[slot] is not None:
            self.meta_events[slot].synchronize()
        # thousands of sequences per micro-batch are normal (a 2-D model's temporal axis): the host side of
        # a step must stay well under the kernels' time, so no Python loop touches the lengths
        row = self.meta_host_np[slot]
        row[0] = 0
        np.cumsum(lens, out=row[1: n + 1])
        used = n + 1
        n_seg = 0
        if seg is not None:
            n_seg = int(seg.shape[0])
            row[used: used + 3 * n_seg] = seg.reshape(-1)
            used += 3 * n_seg
        T = int(row[n])
        self.meta_dev[slot, :used].copy_(self.meta_host[slot, :used], non_blocking=True)
        ev = torch.cuda.Event()
        ev.record()
        self.meta_events[slot] = ev
        cu_dev = self.meta_dev[slot, : n + 1]
        seg_dev = self.meta_dev[slot, n + 1: used] if n_seg else None
        return cu_dev, seg_dev, n_seg, T

    def _attention(self, buf: _Buffers, cu_dev, T: int, max_len: int, recompute: int):
        H = self.H
        q, k, v, g, o = (x[:T] for x in (buf.q, buf.k, buf.v, buf.g, buf.o))
        lse = buf.lse[: H * T].view(H, T)
        binding.dcp_varlen_attn_fwd(q, k, v, cu_dev, max_len, self.causal, out=o, lse=lse, workspace=self.ws)
        if recompute > 0:
            first = (o.clone(), lse.clone()) if self.verify_recompute else None
            binding.dcp_varlen_attn_fwd(q, k, v, cu_dev, max_len, self.causal, out=o, lse=lse, workspace=self.ws)
            if first is not None and not (self.torch.equal(first[0], o) and self.torch.equal(first[1], lse)):
                self.recompute_mismatches += 1
        binding.dcp_varlen_attn_bwd(q, k, v, o, g, lse, cu_dev, max_len, self.causal, dq=buf.dq[:T], dk=buf.dk[:T],
                                    dv=buf.dv[:T], workspace=self.ws)

    def run_micro_batch(self, mb: MicroBatch, batch_tokens: Optional[int] = None) -> int:
        """Enqueue one micro-batch: forward (+ recompute forward) + backward, in place on the batch
        buffers if it has no copy list, else gathered into the staging buffers and scattered back.
        batch_tokens = rows of the batch the micro-batch was cut from (needed for the lse planes)."""
        lens = np.asarray(mb.lengths, dtype=np.int32)
        cu_dev, seg_dev, n_seg, T = self._upload(lens, mb.seg)
        max_len = int(lens.max()) if lens.size else 0
        if mb.seg is None:
            self._attention(self.batch, cu_dev, T, max_len, mb.recompute)
            return T
        if self.stage is None:
            self.stage = _Buffers(self.max_tokens, self.H, self.d, self.device)
        b, s = self.batch, self.stage
        row_bytes = self.H * self.d * 2
        for src, dst in ((b.q, s.q), (b.k, s.k), (b.v, s.v), (b.g, s.g)):
            binding.dcp_copy_segments(src, dst, seg_dev, n_seg, row_bytes)
        self._attention(s, cu_dev, T, max_len, mb.recompute)
        for dst, src in ((b.o, s.o), (b.dq, s.dq), (b.dk, s.dk), (b.dv, s.dv)):
            binding.dcp_copy_segments(src, dst, seg_dev, n_seg, row_bytes, reverse=True)
        Tb = int(batch_tokens)
        binding.dcp_copy_segments(s.lse, b.lse, seg_dev, n_seg, 4, reverse=True, n_planes=self.H,
                                  src_plane_bytes=4 * T, dst_plane_bytes=4 * Tb)
        return T

    def run_batch(self, plan: BatchPlan, batch_tokens: int) -> int:
        """Every micro-batch of a plan over the batch in the first `batch_tokens` rows of the batch
        buffers; results land in the batch buffers in input order (lse as [H, batch_tokens])."""
        return sum(self.run_micro_batch(mb, batch_tokens) for mb in plan.micro_batches)

    def check(self):
        binding.dcp_query_status(self.ws)


class HostPipeline:
    """Steps whose inputs live in pinned host memory and whose results go back to it.

    Two StreamRunners (two sets of device buffers) and three streams: while step i computes, the
    inputs of step i+1 cross to the device and the results of step i-1 cross back, the way a
    training loop prefetches its next batch.  Every step's q, k, v, dO are copied in and its o, lse,
    dq, dk, dv are copied out; only the overlap is added.
    """

    def __init__(self, runners: Sequence[StreamRunner], tokens: int):
        import torch
        self.torch = torch
        self.runners = list(runners)
        if len(self.runners) != 2:
            raise ValueError("the pipeline alternates between exactly two runners")
        r = self.runners[0]
        self.T, self.H = tokens, r.H
        shape = (tokens, r.H, r.d)
        self.host_out = [[torch.empty(shape, dtype=torch.bfloat16).pin_memory() for _ in range(4)] for _ in range(2)]
        self.host_lse = [torch.empty((r.H * tokens,), dtype=torch.float32).pin_memory() for _ in range(2)]
        self.s_in, self.s_out = torch.cuda.Stream(), torch.cuda.Stream()

    def run(self, host_in, step_fn, n_steps: int):
        """host_in: pinned q, k, v, dO.  step_fn(runner) enqueues one step's kernels on the current
        stream.  Returns when everything is enqueued; the current stream ends up waiting for the
        last results to reach the host buffers."""
        torch = self.torch
        T, H = self.T, self.H
        s_comp = torch.cuda.current_stream()
        ev_comp, ev_out = [], []
        for i in range(n_steps):
            r = self.runners[i & 1]
            with torch.cuda.stream(self.s_in):
                if i >= 2:
                    self.s_in.wait_event(ev_comp[i - 2])         # that set's inputs are no longer being read
                for hbuf, dbuf in zip(host_in, (r.q, r.k, r.v, r.g)):
                    dbuf[:T].copy_(hbuf, non_blocking=True)
                ev_in = torch.cuda.Event()
                ev_in.record(self.s_in)
            s_comp.wait_event(ev_in)
            if i >= 2:
                s_comp.wait_event(ev_out[i - 2])                 # that set's results have left
            step_fn(r)
            ev = torch.cuda.Event()
            ev.record(s_comp)
            ev_comp.append(ev)
            with torch.cuda.stream(self.s_out):
                self.s_out.wait_event(ev)
                for hbuf, dbuf in zip(self.host_out[i & 1], (r.o, r.dq, r.dk, r.dv)):
                    hbuf.copy_(dbuf[:T], non_blocking=True)
                self.host_lse[i & 1].copy_(r.lse[: H * T], non_blocking=True)
                ev = torch.cuda.Event()
                ev.record(self.s_out)
                ev_out.append(ev)
        for ev in ev_out[-2:]:
            s_comp.wait_event(ev)
