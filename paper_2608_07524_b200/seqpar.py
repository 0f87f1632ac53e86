"""Sequence-parallel attention over a group of p GPUs (the paper's "sequence parallel size" p_i of
Section 3.2; Section 4.1 names the scheme its experiments use: the head-sharded one, in which an
all-to-all on either side of attention trades the token split for a head split).

Outside attention every rank of the group holds a contiguous slice of the packed tokens with all H
heads.  Attention needs whole sequences, so before it one all-to-all re-shards q, k, v (and dO) to
all T tokens x H/p heads, the single-GPU kernels run on that, and one all-to-all brings o (and dq,
dk, dv) back.  There is no other collective, and no peer memory is touched by any kernel of this
library: the exchanges are torch.distributed calls (NCCL on GPUs, gloo in the CPU tests).

Only host logic and data movement live here; the attention itself is the library's kernels.
"""
from __future__ import annotations

from typing import Callable, List, Optional, Sequence, Tuple


def token_slices(total_tokens: int, p: int) -> List[Tuple[int, int]]:
    """Contiguous token ranges of the p ranks, sizes differing by at most one."""
    if p < 1 or total_tokens < 0:
        raise ValueError("need p >= 1 and total_tokens >= 0")
    base, extra = divmod(total_tokens, p)
    out, start = [], 0
    for r in range(p):
        n = base + (1 if r < extra else 0)
        out.append((start, start + n))
        start += n
    return out


def _group_info(group):
    import torch.distributed as dist
    return dist.get_rank(group), dist.get_world_size(group)


def scatter_heads(x_local, slices: Sequence[Tuple[int, int]], group=None):
    """[t_r, H, d] (this rank's tokens, all heads) -> [T, H/p, d] (all tokens, this rank's heads)."""
    import torch
    import torch.distributed as dist
    rank, p = _group_info(group)
    t_r, H, d = x_local.shape
    if H % p or t_r != slices[rank][1] - slices[rank][0]:
        raise ValueError("heads must divide by the group size and the local slice must match `slices`")
    hp = H // p
    # block j of the send buffer = head group j of the local tokens
    send = x_local.view(t_r, p, hp, d).permute(1, 0, 2, 3).contiguous().view(p * t_r, hp, d)
    sizes = [b - a for a, b in slices]
    recv = torch.empty((sum(sizes), hp, d), dtype=x_local.dtype, device=x_local.device)
    dist.all_to_all_single(recv, send, output_split_sizes=sizes, input_split_sizes=[t_r] * p, group=group)
    return recv


def gather_heads(y, slices: Sequence[Tuple[int, int]], group=None):
    """[T, H/p, d] (all tokens, this rank's heads) -> [t_r, H, d] (this rank's tokens, all heads)."""
    import torch
    import torch.distributed as dist
    rank, p = _group_info(group)
    T, hp, d = y.shape
    sizes = [b - a for a, b in slices]
    if T != sum(sizes):
        raise ValueError("token count does not match `slices`")
    t_r = sizes[rank]
    recv = torch.empty((p * t_r, hp, d), dtype=y.dtype, device=y.device)
    dist.all_to_all_single(recv, y.contiguous(), output_split_sizes=[t_r] * p, input_split_sizes=sizes, group=group)
    return recv.view(p, t_r, hp, d).permute(1, 0, 2, 3).contiguous().view(t_r, p * hp, d)


def sp_attention_fwd(q_local, k_local, v_local, cu_seqlens, max_seqlen: int, causal: bool, total_tokens: int,
                     group=None, attn_fwd: Optional[Callable] = None):
    """Forward over the group.  Returns (o_local [t_r, H, d], ctx); ctx holds the head-sharded
    tensors the backward needs (q, k, v, o as [T, H/p, d] and lse as [H/p, T])."""
    if attn_fwd is None:
        from . import binding
        attn_fwd = binding.dcp_varlen_attn_fwd
    _, p = _group_info(group)
    slices = token_slices(total_tokens, p)
    q, k, v = (scatter_heads(x, slices, group) for x in (q_local, k_local, v_local))
    o, lse = attn_fwd(q, k, v, cu_seqlens, max_seqlen, causal)
    return gather_heads(o, slices, group), (q, k, v, o, lse, slices)


def sp_attention_bwd(do_local, ctx, cu_seqlens, max_seqlen: int, causal: bool, group=None,
                     attn_bwd: Optional[Callable] = None):
    """Backward over the group: (dq, dk, dv), each [t_r, H, d]."""
    if attn_bwd is None:
        from . import binding
        attn_bwd = binding.dcp_varlen_attn_bwd
    q, k, v, o, lse, slices = ctx
    do = scatter_heads(do_local, slices, group)
    dq, dk, dv = attn_bwd(q, k, v, o, do, lse, cu_seqlens, max_seqlen, causal)
    return tuple(gather_heads(x, slices, group) for x in (dq, dk, dv))
