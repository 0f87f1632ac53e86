#!/usr/bin/env python
"""Benchmark of the packed variable-length attention hot path (plan -> forward -> backward).

    python bench.py [--gpus N] [--steps K] [--warmup W]
                    [--workload video|text|extreme|stream|spatial2d|temporal2d] [--order longest|input]
    python bench.py --impl reference ...        # the fp64 CPU oracle on a bounded sample

One step = one pass of the whole path over one synthetic batch: dcp_plan on the batch's lengths,
then for every micro-batch the work-list kernels, forward attention, and the three backward kernels
(plus a second forward when the plan asks for recomputation, and the gather / scatter copies when the
plan splits the batch).  Inputs are resident in HBM before the timed region; they are several times
larger than L2, so no flush is needed between steps.
Prints one JSON line (rank 0).  Under torchrun every rank runs the same batch shape on its own GPU
(weak scaling, no data-path collective); time is the max over ranks.  At one GPU the line also
carries, under "others", a few steps of every other workload, so that one run records them all.
"""
from __future__ import annotations

import argparse
import json
import os
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

METRIC = "varlen_attn_fwd_bwd_tflops"
UNIT = "TFLOP/s"
WORKLOADS = ["video", "text", "extreme", "stream", "spatial2d", "temporal2d"]


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            p = json.load(f)
        return {"burst": float(p["bf16_tflops"]), "sustained": float(p["bf16_tflops_sustained"]),
                "hbm_gbs": float(p["hbm_gbs"]), "source": "measured"}
    except Exception:
        return {"burst": 1590.0, "sustained": 1400.0, "hbm_gbs": 6650.0, "source": "fallback"}


def load_dram_traffic(workload: str):
    """DRAM bytes one backward-main launch moves on this workload, as a profiler capture measured them
    (a small case scaled by tokens where the full one is too large to capture), or None if no capture of
    the current kernel is on record."""
    try:
        with open(os.path.join(ROOT, "profiles", "dram_traffic.json")) as f:
            entry = json.load(f)["bwd_main"].get(workload)
        return float(entry["bytes_per_launch"]) if entry and not entry.get("stale") else None
    except Exception:
        return None


class ClockSampler(threading.Thread):
    """Samples SM clock and throttle reasons of one GPU through NVML while the timed region runs."""
    REASONS = {0x4: "sw_power_cap", 0x8: "hw_slowdown", 0x20: "sw_thermal_slowdown", 0x40: "hw_thermal_slowdown",
               0x80: "hw_power_brake_slowdown"}

    def __init__(self, index: int, period: float = 0.05):
        super().__init__(daemon=True)
        self.index, self.period = index, period
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self._stop_flag = threading.Event()
        self.ok = False
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = int(pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM))
            self.ok = True
        except Exception:
            self.ok = False

    def run(self):
        if not self.ok:
            return
        while not self._stop_flag.is_set():
            try:
                self.samples.append(int(self.nv.nvmlDeviceGetClockInfo(self.h, self.nv.NVML_CLOCK_SM)))
                bits = int(self.nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h))
                for bit, name in self.REASONS.items():
                    if bits & bit:
                        self.reasons.add(name)
            except Exception:
                pass
            time.sleep(self.period)

    def stop(self):
        self._stop_flag.set()
        self.join(timeout=2)
        s = sorted(self.samples)
        return {"sm_mhz": s[len(s) // 2] if s else None, "sm_max_mhz": self.max_mhz,
                "reasons": sorted(self.reasons), "samples": len(s)}


def physical_gpu_index(local_index: int) -> int:
    vis = os.environ.get("CUDA_VISIBLE_DEVICES")
    if vis:
        try:
            return int(vis.split(",")[local_index])
        except Exception:
            return local_index
    return local_index


def workload(name: str):
    from paper_2608_07524_b200 import inputs
    idx = {"text": 2, "video": 3, "extreme": 4}.get(name)
    return inputs.config(idx) if idx else None


# ------------------------------------------------------------------------------------------ oracle arm
def oracle_sample(seq_len: int, n_heads: int, head_dim: int, causal: bool, seed: int = 12):
    """fp64 oracle forward + backward on one synthetic sequence; returns (seconds, counted flops)."""
    import oracle
    from paper_2608_07524_b200 import inputs
    q, k, v, g = inputs.make_qkvg(seq_len, n_heads, head_dim, seed)
    cu = [0, seq_len]
    t0 = time.perf_counter()
    oracle.attn_fwd(q, k, v, cu, causal)
    oracle.attn_bwd(q, k, v, g, cu, causal)
    dt = time.perf_counter() - t0
    flops = 14.0 * seq_len * seq_len * head_dim * n_heads * (0.5 if causal else 1.0)
    return dt, flops


def run_reference(args):
    """The oracle as the reference arm: each step is a bounded sample of the workload."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import oracle
    w = workload(args.workload) or workload("video")
    L = 2048
    sample = f"one {L}-token sequence of the {w.name} workload, {w.n_heads} heads, head_dim {w.head_dim}, fwd+bwd in fp64"
    for _ in range(args.warmup):
        oracle_sample(L, w.n_heads, w.head_dim, w.causal)
    total, flops = 0.0, 0.0
    for _ in range(args.steps):
        dt, f = oracle_sample(L, w.n_heads, w.head_dim, w.causal)
        total += dt
        flops += f
    value = flops / total / 1e12
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": 1e3 * total / args.steps, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": f"{w.name} (bounded sample)", "sample": sample},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": oracle.num_threads(), "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


# ------------------------------------------------------------------------------------------ CUDA arm
class Job:
    """One workload set up for timing: its batches, a runner holding them on the device, and `step`."""

    def __init__(self, args, name: str, dev, rank: int, shuffle: bool = False):
        import numpy as np
        from paper_2608_07524_b200 import inputs
        from paper_2608_07524_b200.stream import StreamRunner
        self.args, self.workload = args, name
        self.axis = None
        if name == "stream":
            self.batches = inputs.stream_batches()[: args.stream_batches]
            self.H, self.d, self.causal = 16, 128, False
            self.desc = (f"stream: {len(self.batches)} batches of the video length mix, Lambda={args.layers}, "
                         f"budget {args.budget_gb} GB")
        elif name in ("spatial2d", "temporal2d"):
            # the paper's second architecture attends along one axis of a clip at a time: the planner sees the
            # clips, the kernels see one sequence per latent frame (spatial) or per spatial position (temporal)
            self.axis = name[:-2]
            clips = inputs.video_clips()
            self.batches, self.H, self.d, self.causal = [[f * s for f, s in clips]], 16, args.head_dim, False
            seqs = inputs.axis_lengths(clips, self.axis)
            self.n_axis_seqs = len(seqs)
            self.desc = (f"config-3 clips, {self.axis} axis of a 2-D model: {len(seqs)} sequences of {min(seqs)}-{max(seqs)} "
                         f"tokens, {sum(seqs)} tokens, 16 heads, head_dim {self.d}, bidirectional")
        else:
            w = workload(name)
            lengths = [L for L in w.lengths if not args.drop_longer_than or L <= args.drop_longer_than]
            if args.longest_last:
                lengths = sorted(lengths)              # the hardest order for a scheduler that takes sequences as they come
            self.batches, self.H, self.d, self.causal = [lengths], w.n_heads, w.head_dim, w.causal
            self.desc = {"video": "config 3 video-DiT-like: 24 sequences, 124992 tokens, 16 heads, head_dim 128, bidirectional",
                         "text": "config 2 text-like: 32 sequences, 79299 tokens, 16 heads, head_dim 128, causal",
                         "extreme": "config 4 extreme imbalance: 131072 + 64 short, 206646 tokens, 8 heads, head_dim 128, causal"}[name]
            if args.drop_longer_than:
                self.desc += f" (profiling subset: sequences longer than {args.drop_longer_than} dropped)"
            if args.longest_last:
                self.desc += " (packed shortest first, the longest sequence last)"
        self.budget = int(args.budget_gb * 10 ** 9)
        self.max_tokens = max(sum(b) for b in self.batches)
        self.max_seqs = max(len(b) for b in self.batches) if self.axis is None else self.n_axis_seqs
        self.value_seed = 12 + 100 * rank
        self.dev = dev
        self.runner = StreamRunner(self.max_tokens, self.max_seqs, self.H, self.d, self.causal, dev, value_seed=self.value_seed)
        self.profile, self.plan_kw = None, {}
        self.np = np

    def use_profile(self):
        # Section 3.5: measure t_f, t_b per length bucket on this GPU (second of two runs) and let the
        # planner use the table instead of its L^2 stand-in; T_C is then in nanoseconds
        from paper_2608_07524_b200.profiler import dual_layer_profile
        buckets = sorted(set(L for b in self.batches for L in b))
        if len(buckets) > 16:
            buckets = [buckets[i * (len(buckets) - 1) // 15] for i in range(16)]
        self.profile = dual_layer_profile(buckets, self.H, self.d, self.causal, device=self.dev)
        self.plan_kw = dict(profile=self.profile, fixed_cost=self.args.fixed_cost_ns)
        self.desc += f", planner fed by a {len(buckets)}-bucket dual-layer profile (T_C = {self.args.fixed_cost_ns} ns)"

    def flops_of(self, lengths):
        ls = self.np.asarray(lengths, dtype=self.np.float64)
        f = 14.0 * float((ls * ls).sum()) * self.d * self.H
        return 0.5 * f if self.causal else f

    def along_axis(self, mb):
        if self.axis is None:
            return mb
        from paper_2608_07524_b200 import inputs
        from paper_2608_07524_b200.stream import MicroBatch
        return MicroBatch(inputs.axis_lengths_array([inputs.clip_shape(int(L)) for L in mb.lengths], self.axis), mb.recompute,
                          mb.seq_index, mb.seg)

    def step(self, r=None):
        from paper_2608_07524_b200.stream import plan_batch
        r = self.runner if r is None else r
        tokens, flops = 0, 0.0
        for lengths in self.batches:
            plan = plan_batch(lengths, self.budget, self.H, self.d, n_layers=self.args.layers, **self.plan_kw)
            batch_tokens = int(sum(lengths))
            for mb in plan.micro_batches:
                mb = self.along_axis(mb)
                tokens += r.run_micro_batch(mb, batch_tokens)
                flops += self.flops_of(mb.lengths)
        return tokens, flops

    def sm_busy(self):
        """Per persistent CTA, how long it was busy in the last forward and backward main launch: the spread
        is the single-GPU imbalance (max / mean = 1 means every SM worked until the end)."""
        from paper_2608_07524_b200 import binding as B
        out = {}
        for which, key in ((0, "fwd"), (1, "bwd_main")):
            try:
                begin, end = B.dcp_read_cta_spans(self.runner.ws, which)
            except B.DcpError:
                continue
            if begin.size == 0:
                continue
            busy = self.np.sort((end - begin).astype(self.np.float64)) / 1e6
            span = float(end.max() - begin.min()) / 1e6
            out[key] = {"ctas": int(busy.size), "min_ms": float(busy[0]), "median_ms": float(busy[busy.size // 2]),
                        "max_ms": float(busy[-1]), "max_over_mean": float(busy[-1] / max(busy.mean(), 1e-12)),
                        "idle_frac": float(1.0 - busy.mean() / max(span, 1e-12))}
        return out


def virtual_rank_balance(dev, world: int = 8, n_global: int = 2):
    """Section 2.3 / 4.2 of the paper on one GPU: the imbalance ratio (slowest rank's time over the mean) of `world`
    data-parallel ranks, with every rank's forward + backward MEASURED on this GPU one after the other.  A global
    step is `world` batches of the stream; `as_drawn` gives rank r batch r, `sharded` deals all their sequences out
    with the library's dcp_shard_sequences (longest first to the least loaded rank, load = L^2)."""
    from paper_2608_07524_b200 import inputs
    from paper_2608_07524_b200.profiler import _gpu_layer
    from paper_2608_07524_b200.shard import shard_sequences, imbalance
    run = _gpu_layer(16, 128, False, dev)
    batches = inputs.stream_batches()[: world * n_global]
    out = {"as_drawn": [], "sharded": [], "sharded_model": []}
    run(batches[0])                                              # warm-up
    for gstep in range(n_global):
        group = batches[gstep * world:(gstep + 1) * world]
        everything = [L for b in group for L in b]
        owned = shard_sequences(everything, world)
        for key, parts in (("as_drawn", group), ("sharded", [[everything[i] for i in idx] for idx in owned])):
            times = [sum(run(list(part))) if part else 0.0 for part in parts]
            out[key].append(max(times) / (sum(times) / len(times)))
        out["sharded_model"].append(imbalance(everything, world))
    return {"workload": f"{n_global} global steps of {world} stream batches (24 sequences each), every rank's fwd + bwd timed on this GPU",
            "ranks": world, "max_over_mean_as_drawn": sum(out["as_drawn"]) / n_global,
            "max_over_mean_sharded": sum(out["sharded"]) / n_global,
            "max_over_mean_sharded_by_the_L2_model": sum(out["sharded_model"]) / n_global}


def timed_steps(job, steps, warmup, barrier):
    """(ms over `steps` steps, tokens, flops, launches, per-kernel profile) after `warmup` untimed steps."""
    import torch
    from paper_2608_07524_b200 import binding as B
    for _ in range(warmup):
        job.step()
    job.runner.check()
    B.dcp_profile_enable(True)
    B.dcp_profile_read()
    barrier()
    launches0 = B.dcp_launch_count()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    tokens = flops = 0
    for _ in range(steps):
        t, f = job.step()
        tokens += t
        flops += f
    e1.record()
    torch.cuda.synchronize()
    ms_total = e0.elapsed_time(e1)
    launches = B.dcp_launch_count() - launches0
    barrier()
    prof = B.dcp_profile_read()
    B.dcp_profile_enable(False)
    job.runner.check()
    return ms_total, tokens, flops, launches, prof


def run_ours(args):
    import torch
    import torch.distributed as dist
    from paper_2608_07524_b200 import binding as B
    from paper_2608_07524_b200.stream import HostPipeline, StreamRunner

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py: no CUDA device; the attention path has no CPU fallback")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)
    B.lib()      # fail loudly here if libdcp.so is missing
    B.dcp_set_work_order(args.order == "input")

    job = Job(args, args.workload, dev, rank)
    if args.plan == "profiled":
        job.use_profile()
    H, d, causal, max_tokens, max_seqs = job.H, job.d, job.causal, job.max_tokens, job.max_seqs
    runner, step, axis, desc = job.runner, job.step, job.axis, job.desc

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    sampler = ClockSampler(physical_gpu_index(local))
    for _ in range(args.warmup):
        step()
    runner.check()
    sampler.start()
    ms_total, tokens, flops, launches, prof = timed_steps(job, args.steps, 0, barrier)
    clocks = sampler.stop()
    sm_busy = job.sm_busy()

    t_ms = torch.tensor([ms_total], dtype=torch.float64, device=dev)
    totals = torch.tensor([flops, float(tokens)], dtype=torch.float64, device=dev)
    if world > 1:
        dist.all_reduce(t_ms, op=dist.ReduceOp.MAX)
        dist.all_reduce(totals, op=dist.ReduceOp.SUM)
    ms_total = float(t_ms.item())
    flops_all, tokens_all = float(totals[0].item()), float(totals[1].item())
    value = flops_all / (ms_total * 1e-3) / 1e12

    # ---- end-to-end: same path with HOST buffers, copies inside the timed region (single-batch workloads)
    def measure_e2e():
        T = max_tokens
        host_in = [torch.empty((T, H, d), dtype=torch.bfloat16).pin_memory() for _ in range(4)]
        for hbuf, dbuf in zip(host_in, (runner.q, runner.k, runner.v, runner.g)):
            hbuf.copy_(dbuf[:T])
        host_out = [torch.empty((T, H, d), dtype=torch.bfloat16).pin_memory() for _ in range(4)]
        host_lse = torch.empty((H * T,), dtype=torch.float32).pin_memory()
        n_e2e = max(1, min(args.steps, 3))

        def e2e_step():
            for hbuf, dbuf in zip(host_in, (runner.q, runner.k, runner.v, runner.g)):
                dbuf[:T].copy_(hbuf, non_blocking=True)
            step()
            for hbuf, dbuf in zip(host_out, (runner.o, runner.dq, runner.dk, runner.dv)):
                hbuf.copy_(dbuf[:T], non_blocking=True)
            host_lse.copy_(runner.lse[: H * T], non_blocking=True)

        e2e_step()
        barrier()
        s0, s1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        s0.record()
        for _ in range(n_e2e):
            e2e_step()
        s1.record()
        torch.cuda.synchronize()
        serial_ms = torch.tensor([s0.elapsed_time(s1)], dtype=torch.float64, device=dev)

        # The same with two sets of device buffers and three streams: while step i computes, the inputs of
        # step i+1 arrive and the results of step i-1 leave (a training loop prefetches its next batch the
        # same way).  Every step's inputs still cross PCIe and every step's results are read back; the
        # timed region includes filling and draining the pipeline.
        runners = [runner, StreamRunner(max_tokens, max_seqs, H, d, causal, dev, value_seed=13 + 100 * rank)]
        pipe = HostPipeline(runners, T)
        # long enough that filling and draining the pipeline (one step's copies in, one step's out) is a small part
        n_pipe = min(max(4 * n_e2e, 2 * args.steps), 40)

        def pipeline(n):
            pipe.run(host_in, step, n)

        pipeline(2)
        barrier()
        s0, s1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        s0.record()
        pipeline(n_pipe)
        s1.record()
        torch.cuda.synchronize()
        e2e_ms = torch.tensor([s0.elapsed_time(s1)], dtype=torch.float64, device=dev)
        if world > 1:
            dist.all_reduce(e2e_ms, op=dist.ReduceOp.MAX)
            dist.all_reduce(serial_ms, op=dist.ReduceOp.MAX)
        for r in runners:
            r.check()
        per_step_flops = flops_all / args.steps
        h2d = 4 * T * H * d * 2
        d2h = 4 * T * H * d * 2 + 4 * H * T
        e2e = {"value": per_step_flops * n_pipe / (float(e2e_ms.item()) * 1e-3) / 1e12, "unit": UNIT,
               "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h, "steps": n_pipe,
               "how": "two sets of device buffers, copies and compute on three streams",
               "one_stream_value": per_step_flops * n_e2e / (float(serial_ms.item()) * 1e-3) / 1e12}
        del runners, pipe
        del host_in, host_out, host_lse
        return e2e

    e2e = None
    if args.workload != "stream":
        if world > 1:
            e2e = measure_e2e()          # every rank must reach the same collectives
        else:
            try:
                e2e = measure_e2e()
            except Exception as ex:      # e.g. pinned host memory refused: keep the device-timed line
                print(f"bench.py: end-to-end leg failed: {ex}", file=sys.stderr)
                e2e = {"value": None, "unit": UNIT, "error": str(ex)[:200]}

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    peaks = load_peaks()
    bwd_ms, bwd_n = prof["bwd_main"]
    bwd_flops_per_launch = (flops / args.steps) * (2.5 / 3.5) / max(bwd_n / args.steps, 1)
    achieved = bwd_flops_per_launch / (bwd_ms / max(bwd_n, 1) * 1e-3) / 1e12 if bwd_n else None
    plain = not args.drop_longer_than and args.layers == 1 and not args.longest_last and args.order == "longest"
    roofline = {"bound": "tensor", "kernel": "attn_bwd_kernel (backward main)", "achieved": achieved,
                "peak": peaks["sustained"], "unit": UNIT, "frac": (achieved / peaks["sustained"]) if achieved else None,
                "peak_source": f"bf16_tflops_sustained of {peaks['source']} MEASURED_PEAKS.json",
                "traffic": load_dram_traffic(args.workload) if plain else None,
                "launches": bwd_n, "avg_launch_ms": bwd_ms / max(bwd_n, 1)}
    if axis == "temporal" and bwd_n:
        # sequences of 1-13 tokens run on the short-sequence kernels, which are bound by HBM.  Algorithmic bytes of
        # the backward kernel per (token, head): q, k, v, dO read and dq, dk, dv written (7 d bf16), lse read (4);
        # D is formed in registers and o is not read.
        tok_per_launch = tokens_all / world / max(bwd_n, 1)
        gbs = tok_per_launch * H * (7 * d * 2 + 4) / (bwd_ms / bwd_n * 1e-3) / 1e9
        roofline = {"bound": "hbm", "kernel": "small_attn_kernel (backward, short sequences)", "achieved": gbs,
                    "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": gbs / peaks["hbm_gbs"],
                    "peak_source": f"hbm_gbs of {peaks['source']} MEASURED_PEAKS.json",
                    "traffic": load_dram_traffic("temporal2d") if d == 128 else None,
                    "launches": bwd_n, "avg_launch_ms": bwd_ms / bwd_n}

    # ---- a few steps of every other workload, so that one run records them all (single GPU only)
    others = None
    if world == 1 and not args.no_others:
        others = {}
        del job, runner, step
        torch.cuda.empty_cache()
        # every other workload at head_dim 128, and the two axes of the 2-D model at the paper's own width (72)
        for key, name, width in [(n, n, 128) for n in WORKLOADS] + [("spatial2d_d72", "spatial2d", 72), ("temporal2d_d72", "temporal2d", 72)]:
            if name == args.workload and width == args.head_dim:
                continue
            o_args = argparse.Namespace(**vars(args))
            o_args.drop_longer_than, o_args.longest_last = 0, False
            o_args.layers, o_args.budget_gb, o_args.stream_batches, o_args.head_dim = 1, 180.0, 32, width
            try:
                oj = Job(o_args, name, dev, rank)
                n_steps = 2 if name in ("stream", "extreme") else 5
                ms, tok, fl, _, pr = timed_steps(oj, n_steps, 3 if name != "stream" else 1, barrier)
                v = fl / (ms * 1e-3) / 1e12
                others[key] = {"workload": oj.desc, "steps": n_steps, "ms_per_step": ms / n_steps, "value": v, "unit": UNIT,
                                "tokens_per_s": tok / (ms * 1e-3), "frac_of_bf16_peak_burst": v / peaks["burst"],
                                "kernel_ms_per_step": {k: x[0] / n_steps for k, x in pr.items()},
                                "sm_busy": oj.sm_busy()}
                del oj
            except Exception as ex:
                others[key] = {"error": str(ex)[:200]}
            torch.cuda.empty_cache()
        try:
            others["balance_w8"] = virtual_rank_balance(dev)
        except Exception as ex:
            others["balance_w8"] = {"error": str(ex)[:200]}
        torch.cuda.empty_cache()

    cpu_baseline = None
    if world == 1 and not args.no_cpu_baseline:
        import oracle
        Ls = 3600
        dt, f = oracle_sample(Ls, H, d, causal)
        cpu_baseline = {"value": f / dt / 1e12, "unit": UNIT, "cores": oracle.num_threads(), "kind": "oracle",
                        "sample": f"one {Ls}-token sequence, {H} heads, head_dim {d}, fwd+bwd in fp64, {dt:.1f} s"}

    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": ms_total / args.steps, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16", "data": "synthetic",
        "config": {"workload": desc, "l2": "inputs (2 GB+) larger than L2, no flush",
                   "hbm_budget_bytes": int(args.budget_gb * 10 ** 9), "n_layers": args.layers, "work_order": args.order},
        "tokens_per_s": tokens_all / (ms_total * 1e-3),
        "frac_of_bf16_peak": {"burst": value / world / peaks["burst"], "sustained": value / world / peaks["sustained"],
                              "source": peaks["source"]},
        "kernel_ms_per_step": {k: v[0] / args.steps for k, v in prof.items()},
        "sm_busy": sm_busy,
        "clocks": clocks, "e2e": e2e, "gpu_launches": launches, "roofline": roofline, "cpu_baseline": cpu_baseline,
        "others": others,
    }
    print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


def run_uniform(args):
    """Not the contract line: one JSON line per sequence length for batches of equal sequences (131072 tokens, 16
    heads of --head-dim, bidirectional), forward + backward, with the per-kernel times.  It shows where the paths
    change (short-sequence kernels up to 32 tokens, one tile per sequence up to 128, work items of growing
    length after that) and what each costs against the HBM and tensor rooflines."""
    import torch
    from paper_2608_07524_b200 import binding as B
    dev, H, d, total = "cuda:0", 16, args.head_dim, 131072
    torch.cuda.set_device(0)
    for L in [int(x) for x in args.uniform.split(",")]:
        n = max(1, total // L)
        T = n * L
        cu = torch.arange(0, T + 1, L, dtype=torch.int32, device=dev)
        q, k, v, g = (torch.randn(T, H, d, device=dev, dtype=torch.bfloat16) for _ in range(4))
        ws = B.alloc_workspace(T, n, H, d, True, dev)
        o, dq, dk, dv = (torch.empty_like(q) for _ in range(4))
        lse = torch.empty(H, T, device=dev)

        def step():
            B.dcp_varlen_attn_fwd(q, k, v, cu, L, False, 0.0, out=o, lse=lse, workspace=ws)
            B.dcp_varlen_attn_bwd(q, k, v, o, g, lse, cu, L, False, 0.0, dq=dq, dk=dk, dv=dv, workspace=ws)

        for _ in range(max(args.warmup, 3)):
            step()
        B.dcp_query_status(ws)
        B.dcp_profile_enable(True)
        B.dcp_profile_read()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(args.steps):
            step()
        e1.record()
        torch.cuda.synchronize()
        prof = B.dcp_profile_read()
        B.dcp_profile_enable(False)
        ms = e0.elapsed_time(e1) / args.steps
        print(json.dumps({"uniform_tokens_per_sequence": L, "sequences": n, "tokens": T, "heads": H, "head_dim": d,
                          "ms_per_step": ms, "tflops": 14.0 * n * L * L * d * H / (ms * 1e-3) / 1e12,
                          "algorithmic_gb_per_s": T * H * (12 * d * 2 + 12) / (ms * 1e-3) / 1e9,
                          "kernel_ms_per_step": {k_: x[0] / args.steps for k_, x in prof.items()}}), flush=True)
        del q, k, v, g, o, dq, dk, dv, lse, ws
        torch.cuda.empty_cache()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=10)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="video", choices=WORKLOADS)
    ap.add_argument("--head-dim", type=int, default=128,
                    help="head dimension of the 2-D workloads (the paper's second model has 72)")
    ap.add_argument("--stream-batches", type=int, default=256)
    ap.add_argument("--layers", type=int, default=1, help="planner's layer count Lambda")
    ap.add_argument("--plan", default="model", choices=["model", "profiled"],
                    help="planner's forward-time source: the L^2 model or a dual-layer profile measured first")
    ap.add_argument("--fixed-cost-ns", type=int, default=20000, help="T_C per micro-batch for --plan profiled")
    ap.add_argument("--budget-gb", type=float, default=180.0, help="planner's HBM budget in decimal GB")
    ap.add_argument("--order", default="longest", choices=["longest", "input"],
                    help="work order of the kernels: longest sequence first (the default) or as the sequences come")
    ap.add_argument("--longest-last", action="store_true",
                    help="pack the batch shortest first (with --order input: what the length-aware order is worth)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-others", action="store_true", help="skip the short runs of the other workloads")
    ap.add_argument("--drop-longer-than", type=int, default=0,
                    help="profiling aid: drop sequences longer than this from the workload (0 = keep all)")
    ap.add_argument("--uniform", default="", metavar="L[,L...]",
                    help="instead of the contract line: batches of equal sequences of these lengths, one JSON line each")
    args = ap.parse_args()
    if args.uniform:
        run_uniform(args)
    elif args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
