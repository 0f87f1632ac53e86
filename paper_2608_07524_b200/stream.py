"""Host loop of the end-to-end stream: plan a batch, then run every micro-batch through the kernels.

Per batch (Section 3.1 of the paper: settings are re-chosen for every incoming batch):
    dcp_plan(lengths, budget)  ->  micro-batches (gradient-accumulation steps) and recompute counts
    for each micro-batch:      forward; forward again if its recompute count > 0 (activation
                               recomputation re-runs the layer's forward before its backward,
                               Section 3.4); backward.
All arithmetic happens in libdcp; this module only slices buffers and issues calls.
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import List, Sequence

import numpy as np

from . import binding


@dataclass
class MicroBatch:
    lengths: Sequence[int]    # in planner order (longest first); a list or an integer numpy array
    recompute: int            # layers whose forward is re-run before backward

    @property
    def total_tokens(self) -> int:
        return int(sum(self.lengths)) if isinstance(self.lengths, list) else int(self.lengths.sum())


def plan_batch(lengths: Sequence[int], hbm_budget_bytes: int, n_heads: int, head_dim: int,
               n_layers: int = 1, fixed_cost: int = 1 << 24, profile=None) -> List[MicroBatch]:
    """Micro-batches of one batch.  With `profile` (a profiler.ProfileTable) the per-layer forward
    time of every sequence comes from the measured table (Section 3.5) and fixed_cost is in
    nanoseconds; without it the planner uses its L^2 stand-in and fixed_cost is in its units."""
    if profile is None:
        mb_id, recompute, _ = binding.dcp_plan(lengths, hbm_budget_bytes, n_heads=n_heads, head_dim=head_dim,
                                               n_layers=n_layers, fixed_cost=fixed_cost)
    else:
        fwd_time = [profile.fwd_time(int(L)) for L in lengths]
        mb_id, recompute, _ = binding.dcp_plan_profiled(lengths, fwd_time, hbm_budget_bytes, n_heads=n_heads,
                                                        head_dim=head_dim, n_layers=n_layers, fixed_cost=fixed_cost)
    out = [MicroBatch([], r) for r in recompute]
    # inside a micro-batch keep the planner's order: longest first, ties by input index
    for i in sorted(range(len(lengths)), key=lambda i: (-lengths[i], i)):
        out[mb_id[i]].lengths.append(int(lengths[i]))
    return out


class StreamRunner:
    """Runs micro-batches out of pre-allocated device buffers sized for the largest micro-batch.

    The synthetic stream reuses the first `tokens` rows of the q/k/v/dO buffers for every
    micro-batch (the values are random either way); outputs go to preallocated tensors.
    """

    def __init__(self, max_tokens: int, max_seqs: int, n_heads: int, head_dim: int, causal: bool, device,
                 value_seed: int = 20):
        import torch
        from . import inputs
        self.torch = torch
        self.H, self.d, self.causal, self.device = n_heads, head_dim, causal, device
        self.q, self.k, self.v, self.g = inputs.make_qkvg_device(max_tokens, n_heads, head_dim, value_seed, device)
        self.o = torch.empty_like(self.q)
        self.dq, self.dk, self.dv = (torch.empty_like(self.q) for _ in range(3))
        self.lse = torch.empty(n_heads * max_tokens, dtype=torch.float32, device=device)
        _, bwd_bytes = binding.dcp_varlen_attn_workspace(max_tokens, max_seqs, n_heads, head_dim)
        self.ws = torch.empty(bwd_bytes, dtype=torch.uint8, device=device)
        # cu_seqlens travel through a small ring of pinned host / device slots; a slot is reused
        # only after the copy that read it has finished (tracked by an event per slot)
        self.n_slots = 16
        self.cu_host = torch.empty((self.n_slots, max_seqs + 1), dtype=torch.int32).pin_memory()
        self.cu_host_np = self.cu_host.numpy()          # same memory: boundaries are written with numpy
        self.cu_dev = torch.empty((self.n_slots, max_seqs + 1), dtype=torch.int32, device=device)
        self.cu_events = [None] * self.n_slots
        self.calls = 0

    def run_micro_batch(self, mb: MicroBatch) -> int:
        """Enqueue forward (+ recompute forward) + backward for one micro-batch; returns its tokens."""
        torch = self.torch
        lens = np.asarray(mb.lengths, dtype=np.int32)
        n = int(lens.size)
        slot = self.calls % self.n_slots
        self.calls += 1
        if self.cu_events[slot] is not None:
            self.cu_events[slot].synchronize()
        # thousands of sequences per micro-batch are normal (a 2-D model's temporal axis): the host side of
        # a step must stay well under the kernels' time, so no Python loop touches the lengths
        cu_np = self.cu_host_np[slot, : n + 1]
        cu_np[0] = 0
        np.cumsum(lens, out=cu_np[1:])
        T = int(cu_np[n])
        cu = self.cu_host[slot, : n + 1]
        cu_dev = self.cu_dev[slot, : n + 1]
        cu_dev.copy_(cu, non_blocking=True)
        ev = torch.cuda.Event()
        ev.record()
        self.cu_events[slot] = ev
        q, k, v, g, o = (x[:T] for x in (self.q, self.k, self.v, self.g, self.o))
        lse = self.lse[: self.H * T].view(self.H, T)
        max_len = int(lens.max())
        for _ in range(1 + (1 if mb.recompute > 0 else 0)):
            binding.dcp_varlen_attn_fwd(q, k, v, cu_dev, max_len, self.causal, out=o, lse=lse, workspace=self.ws)
        binding.dcp_varlen_attn_bwd(q, k, v, o, g, lse, cu_dev, max_len, self.causal, dq=self.dq[:T], dk=self.dk[:T],
                                    dv=self.dv[:T], workspace=self.ws)
        return T

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

