"""Seeded synthetic workloads: sequence-length mixes and bf16 tensor values.

This module holds no attention or planner arithmetic.  It is the one piece that both the CUDA
path's tests and the CPU oracle's tests draw their inputs from, so that both see identical bits.

Length mixes (stand-ins for the paper's data, whose histograms are figures only: the video
length distribution of Section 2.1 and the three synthetic mixes of Appendix A):

  config 1  "tiny"     fixed lengths [17, 64, 100, 255]; 2 heads, head_dim 64; both masks
  config 2  "text"     32 lengths, log-uniform in [512, 8192); 16 heads, head_dim 128; causal
  config 3  "video"    24 lengths ceil(frames/4) * (H/16) * (W/16) with the resolution drawn from
                       {256x256, 480x640, 720x1280} and frames from {1, 16, 32, 51}, weighted
                       toward short clips; 16 heads, head_dim 128; bidirectional
  config 4  "extreme"  one 131072-token sequence plus 64 lengths uniform in [128, 2048];
                       8 heads, head_dim 128; causal
  config 5  "stream"   256 batches, each 24 draws of the config-3 rule from one generator
  "short2d"            the config-3 clips seen by a model that attends along one axis at a time
                       (the paper's second architecture): per latent frame over its 256-3600
                       tokens, then per spatial position over its 1-13 latent frames

Uniform variates come from SplitMix64 so the draws are reproducible in any language.  The
lists for configs 2-4 are also stored as text under tests/golden/ and a test checks that this
module regenerates them.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field
from typing import List

_MASK = (1 << 64) - 1


class SplitMix64:
    """Counter-based 64-bit generator; seed 0 yields 0xe220a8397b1dcdaf first."""

    def __init__(self, seed: int):
        self.state = seed & _MASK

    def next_u64(self) -> int:
        self.state = (self.state + 0x9E3779B97F4A7C15) & _MASK
        z = self.state
        z = ((z ^ (z >> 30)) * 0xBF58476D1CE4E5B9) & _MASK
        z = ((z ^ (z >> 27)) * 0x94D049BB133111EB) & _MASK
        return z ^ (z >> 31)

    def uniform(self) -> float:
        """u in [0, 1) with 53 random bits."""
        return (self.next_u64() >> 11) * (1.0 / (1 << 53))


def text_lengths(n: int = 32, seed: int = 2) -> List[int]:
    g = SplitMix64(seed)
    return [int(math.floor(512.0 * 16.0 ** g.uniform())) for _ in range(n)]


_RES = ((0.5, 256, 256), (0.8, 480, 640), (1.01, 720, 1280))
_FRAMES = ((0.4, 1), (0.7, 16), (0.9, 32), (1.01, 51))


def _video_sample(g: SplitMix64):
    """(latent frames, tokens per latent frame) of one clip."""
    u1, u2 = g.uniform(), g.uniform()
    h, w = next((hh, ww) for t, hh, ww in _RES if u1 < t)
    frames = next(f for t, f in _FRAMES if u2 < t)
    return -(-frames // 4), (h // 16) * (w // 16)


def _video_draw(g: SplitMix64) -> int:
    f, s = _video_sample(g)
    return f * s


def video_lengths(n: int = 24, seed: int = 3) -> List[int]:
    g = SplitMix64(seed)
    return [_video_draw(g) for _ in range(n)]


def video_clips(n: int = 24, seed: int = 3):
    """The config-3 draws as (latent frames, tokens per latent frame) pairs."""
    g = SplitMix64(seed)
    return [_video_sample(g) for _ in range(n)]


def clip_shape(length: int):
    """(latent frames, tokens per frame) of a clip given its token count (the products are distinct)."""
    for _, h, w in _RES:
        for _, frames in _FRAMES:
            f, s = -(-frames // 4), (h // 16) * (w // 16)
            if f * s == length:
                return f, s
    raise ValueError(f"{length} is not a clip length of the video mix")


def axis_lengths(clips, axis: str) -> List[int]:
    """Sequences a 2-D model attends over (one axis at a time): `spatial` gives one sequence per
    latent frame (its tokens attend to each other), `temporal` one sequence per spatial position
    (its frames attend to each other).  Both hold the same tokens in total."""
    if axis not in ("spatial", "temporal"):
        raise ValueError("axis must be 'spatial' or 'temporal'")
    out: List[int] = []
    for f, s in clips:
        out += [s] * f if axis == "spatial" else [f] * s
    return out


def axis_lengths_array(clips, axis: str):
    """axis_lengths as an int32 numpy array, without a Python loop over the sequences."""
    import numpy as np
    if axis not in ("spatial", "temporal"):
        raise ValueError("axis must be 'spatial' or 'temporal'")
    f = np.fromiter((c[0] for c in clips), dtype=np.int32, count=len(clips))
    s = np.fromiter((c[1] for c in clips), dtype=np.int32, count=len(clips))
    return np.repeat(s, f) if axis == "spatial" else np.repeat(f, s)


def short2d_lengths(axis: str, n: int = 24, seed: int = 3) -> List[int]:
    """axis_lengths of the config-3 clips."""
    return axis_lengths(video_clips(n, seed), axis)


def extreme_lengths(n_short: int = 64, seed: int = 4, long_len: int = 131072) -> List[int]:
    g = SplitMix64(seed)
    return [long_len] + [128 + int(math.floor(g.uniform() * 1921.0)) for _ in range(n_short)]


def stream_batches(n_batches: int = 256, per_batch: int = 24, seed: int = 5) -> List[List[int]]:
    g = SplitMix64(seed)
    return [[_video_draw(g) for _ in range(per_batch)] for _ in range(n_batches)]


@dataclass
class Workload:
    name: str
    lengths: List[int]
    n_heads: int
    head_dim: int
    causal: bool
    value_seed: int          # q, k, v, dO use value_seed + 0..3
    cu_seqlens: List[int] = field(init=False)

    def __post_init__(self):
        cu = [0]
        for L in self.lengths:
            cu.append(cu[-1] + int(L))
        self.cu_seqlens = cu

    @property
    def total_tokens(self) -> int:
        return self.cu_seqlens[-1]

    @property
    def max_seqlen(self) -> int:
        return max(self.lengths) if self.lengths else 0

    def fwd_flops(self) -> float:
        """4 * sum(L^2) * d * H, halved under a causal mask (the usual counting convention)."""
        f = 4.0 * sum(float(L) * L for L in self.lengths) * self.head_dim * self.n_heads
        return f * 0.5 if self.causal else f

    def fwd_bwd_flops(self) -> float:
        return 3.5 * self.fwd_flops()


def config(idx: int, causal: bool | None = None) -> Workload:
    """The benchmark's named configurations 1-4 (config 5 is a stream of config-3-like batches)."""
    if idx == 1:
        return Workload("tiny", [17, 64, 100, 255], 2, 64, bool(causal), 4)
    if idx == 2:
        return Workload("text", text_lengths(), 16, 128, True if causal is None else causal, 8)
    if idx == 3:
        return Workload("video", video_lengths(), 16, 128, False if causal is None else causal, 12)
    if idx == 4:
        return Workload("extreme", extreme_lengths(), 8, 128, True if causal is None else causal, 16)
    raise ValueError("config index must be 1..4")


def make_qkvg(total_tokens: int, n_heads: int, head_dim: int, value_seed: int, device="cpu"):
    """q, k, v, dO ~ N(0,1): drawn in fp32 by a seeded CPU generator, rounded to bf16, then moved.
    The same call therefore gives the same bits on every machine and for every device."""
    import torch
    out = []
    for i in range(4):
        gen = torch.Generator(device="cpu")
        gen.manual_seed(value_seed + i)
        x = torch.randn((total_tokens, n_heads, head_dim), generator=gen, dtype=torch.float32)
        out.append(x.to(torch.bfloat16).to(device))
    return out


def make_qkvg_device(total_tokens: int, n_heads: int, head_dim: int, value_seed: int, device):
    """Same distribution drawn directly on `device` (for full-size timing runs, where a CPU draw
    of several GB would dominate the run).  Bits differ from make_qkvg; sampled-row checks pull
    the tensors back to the host instead of regenerating them."""
    import torch
    out = []
    for i in range(4):
        gen = torch.Generator(device=device)
        gen.manual_seed(value_seed + i)
        x = torch.randn((total_tokens, n_heads, head_dim), generator=gen, dtype=torch.float32,
                        device=device)
        out.append(x.to(torch.bfloat16))
        del x
    return out
