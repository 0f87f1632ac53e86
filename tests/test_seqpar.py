"""Sequence-parallel attention (head-sharded, an all-to-all on either side): the exchange and the
composition on two gloo ranks on CPU, with the oracle standing in for the attention kernels; on a
GPU, a group of one rank through the real kernels."""
import os
import socket

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2608_07524_b200 import inputs
from paper_2608_07524_b200.seqpar import (gather_heads, scatter_heads, sp_attention_bwd, sp_attention_fwd,
                                          token_slices)


def test_token_slices():
    assert token_slices(10, 3) == [(0, 4), (4, 7), (7, 10)]
    assert token_slices(2, 4) == [(0, 1), (1, 2), (2, 2), (2, 2)]
    assert token_slices(0, 2) == [(0, 0), (0, 0)]
    with pytest.raises(ValueError):
        token_slices(5, 0)


LENGTHS = [5, 17, 1, 30, 8]          # 61 tokens: an uneven split over two ranks
H, D = 4, 8


def _oracle_fwd(q, k, v, cu, max_seqlen, causal):
    import oracle
    O, L = oracle.attn_fwd(q, k, v, cu, causal)
    return torch.from_numpy(O).to(torch.bfloat16), torch.from_numpy(L).float()


def _oracle_bwd(q, k, v, o, do, lse, cu, max_seqlen, causal):
    import oracle
    return tuple(torch.from_numpy(x).to(torch.bfloat16) for x in oracle.attn_bwd(q, k, v, do, cu, causal))


def _worker(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    cu = np.concatenate([[0], np.cumsum(LENGTHS)]).astype(np.int32)
    T = int(cu[-1])
    q, k, v, g = inputs.make_qkvg(T, H, D, 31)
    a, b = token_slices(T, world)[rank]
    slices = token_slices(T, world)
    # the exchange alone: every rank ends up with all tokens of its heads, and the inverse restores the slice
    qs = scatter_heads(q[a:b].contiguous(), slices)
    hp = H // world
    ok_scatter = torch.equal(qs, q[:, rank * hp:(rank + 1) * hp])
    ok_round = torch.equal(gather_heads(qs, slices), q[a:b])
    res = {}
    for causal in (False, True):
        o_loc, ctx = sp_attention_fwd(q[a:b].contiguous(), k[a:b].contiguous(), v[a:b].contiguous(), cu, max(LENGTHS),
                                      causal, T, attn_fwd=_oracle_fwd)
        dq, dk, dv = sp_attention_bwd(g[a:b].contiguous(), ctx, cu, max(LENGTHS), causal, attn_bwd=_oracle_bwd)
        res[causal] = (o_loc, dq, dk, dv)
    out.put((rank, ok_scatter, ok_round, (a, b), {c: tuple(x.float().numpy() for x in r) for c, r in res.items()}))
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_compose_to_the_single_device_result():
    import oracle
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    got = [out.get(timeout=180) for _ in range(2)]
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    cu = np.concatenate([[0], np.cumsum(LENGTHS)]).astype(np.int32)
    q, k, v, g = inputs.make_qkvg(int(cu[-1]), H, D, 31)
    for rank, ok_scatter, ok_round, (a, b), res in got:
        assert ok_scatter and ok_round
        for causal in (False, True):
            O, _ = oracle.attn_fwd(q, k, v, cu, causal)
            ref = (O,) + tuple(oracle.attn_bwd(q, k, v, g, cu, causal))
            for x, r in zip(res[causal], ref):
                want = torch.from_numpy(r[a:b]).to(torch.bfloat16).float().numpy()     # the stand-in rounds to bf16
                assert x.shape == want.shape and np.array_equal(x, want)


@pytest.mark.gpu
def test_group_of_one_runs_the_kernels():
    from paper_2608_07524_b200 import binding as B
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    os.environ["MASTER_ADDR"], os.environ["MASTER_PORT"] = "127.0.0.1", str(port)
    dist.init_process_group("nccl", rank=0, world_size=1, device_id=torch.device("cuda", 0))
    try:
        lengths = [300, 77, 1000]
        cu = np.concatenate([[0], np.cumsum(lengths)]).astype(np.int32)
        T = int(cu[-1])
        q, k, v, g = (x.cuda() for x in inputs.make_qkvg(T, 4, 128, 33))
        cud = torch.tensor(cu, device="cuda")
        o_sp, ctx = sp_attention_fwd(q, k, v, cud, max(lengths), True, T)
        dq_sp, dk_sp, dv_sp = sp_attention_bwd(g, ctx, cud, max(lengths), True)
        o, lse = B.dcp_varlen_attn_fwd(q, k, v, cud, max(lengths), True)
        dq, dk, dv = B.dcp_varlen_attn_bwd(q, k, v, o, g, lse, cud, max(lengths), True)
        assert torch.equal(o_sp, o) and torch.equal(dk_sp, dk) and torch.equal(dv_sp, dv)
        assert float((dq_sp.float() - dq.float()).abs().max()) <= 2e-2      # atomics: summation order is free
    finally:
        dist.destroy_process_group()
