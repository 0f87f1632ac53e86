"""Sequence-parallel attention over a group of p GPUs (the paper's "sequence parallel size" p_i of
Section 3.2; Section 4.1 names the scheme its experiments use: the head-sharded one, in which an
all-to-all on either side of attention trades the token split for a head split).

Outside attention every rank of the group holds a contiguous slice of the packed tokens with all H
heads.  Attention needs whole sequences, so before it one all-to-all re-shards q, k, v (and dO) to
all T tokens x H/p heads, the single-GPU kernels run on that, and one all-to-all brings o (and dq,
dk, dv) back.  There is no other collective, and no peer memory is touched by any kernel of this
library: the exchanges are torch.distributed calls (NCCL on GPUs, gloo in the CPU tests).

Only host logic and data movement live here; the attention itself is the library's kernels.

Two forms: the first re-shards with a library all-to-all around the unchanged kernels
(scatter_heads / gather_heads / sp_attention_fwd / sp_attention_bwd); the second, at the end of this file,
needs no all-to-all at all: the kernels work in place on token-sharded tensors that every rank has mapped
into one address range (vmm.py) and fetch each tile from its owner when they need it.
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


# ---- the same scheme without materialising the all-to-all ---------------------------------------------------------------
#
# When the token-sharded tensors of the group live in one address range on every rank (vmm.py: each rank maps
# its own slice and its peers' slices back to back), rank r can run attention for its heads [r H/p, (r+1) H/p)
# directly on those tensors: the strided entry points read every tile from wherever it lives (plain TMA loads,
# no multicast) and write o / dq / dk / dv rows straight into their owners' slices.  Nothing is re-sharded and
# no collective moves data; the ranks only have to agree on WHEN: inputs complete before anyone reads them,
# outputs complete before anyone uses them.  `fence` is that agreement - a device synchronise followed by a
# barrier of the group on multiple GPUs, nothing at all for virtual ranks run one after the other on one GPU.

def head_group(rank: int, p: int, n_heads: int) -> slice:
    """Heads that rank `rank` of `p` computes."""
    if n_heads % p or not 0 <= rank < p:
        raise ValueError("heads must divide by the group size and the rank must lie in the group")
    hp = n_heads // p
    return slice(rank * hp, (rank + 1) * hp)


def group_fence(group=None):
    """Everything this rank has enqueued is done, and every rank of the group has said the same."""
    import torch
    import torch.distributed as dist
    torch.cuda.synchronize()
    dist.barrier(group)


def sp_attention_fwd_mapped(q, k, v, o, cu_seqlens, max_seqlen: int, causal: bool, rank: int, p: int,
                            fence: Optional[Callable[[], None]] = None, workspace=None):
    """Forward of rank `rank` on mapped token-sharded tensors q, k, v, o [T, H, d] (all ranks pass views of
    the same memory).  Returns lse [H/p, T] of this rank's heads (rank-local)."""
    from . import binding
    hs = head_group(rank, p, q.shape[1])
    if fence is not None:
        fence()                       # every slice of q, k, v is complete
    _, lse = binding.dcp_varlen_attn_fwd_strided(q[:, hs], k[:, hs], v[:, hs], cu_seqlens, max_seqlen, causal, o[:, hs],
                                                 workspace=workspace)
    if fence is not None:
        fence()                       # every head group of o is complete
    return lse


def sp_attention_bwd_mapped(q, k, v, o, d_o, lse, dq, dk, dv, cu_seqlens, max_seqlen: int, causal: bool, rank: int, p: int,
                            fence: Optional[Callable[[], None]] = None, workspace=None):
    """Backward of rank `rank` on mapped token-sharded tensors; dq, dk, dv [T, H, d] receive this rank's heads."""
    from . import binding
    hs = head_group(rank, p, q.shape[1])
    if fence is not None:
        fence()                       # every slice of dO is complete
    binding.dcp_varlen_attn_bwd_strided(q[:, hs], k[:, hs], v[:, hs], o[:, hs], d_o[:, hs], lse, cu_seqlens, max_seqlen,
                                        causal, dq[:, hs], dk[:, hs], dv[:, hs], workspace=workspace)
    if fence is not None:
        fence()
