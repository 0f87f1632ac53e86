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


def test_granule_aligned_token_slices():
    from paper_2608_07524_b200 import vmm
    gran, row = 2 << 20, 16 * 128 * 2                     # 512 tokens per granule
    r = vmm.token_slices(3000, 4, row, gran)
    assert r == [(0, 1024), (1024, 2048), (2048, 2560), (2560, 3000)]
    assert vmm.slice_bytes(r, row, gran) == [2 * gran, 2 * gran, gran, gran]
    # fewer granules than ranks: trailing ranks get nothing
    assert vmm.token_slices(600, 4, row, gran) == [(0, 512), (512, 600), (600, 600), (600, 600)]
    assert vmm.slice_bytes([(600, 600)], row, gran) == [0]
    # a row that does not divide the granule: boundaries fall where both do
    assert vmm.token_slices(100000, 2, 3 * 1024, 2 << 20)[0][1] % 2048 == 0
    for T in (0, 1, 511, 512, 513, 70000):
        for p in (1, 2, 3, 8):
            rs = vmm.token_slices(T, p, row, gran)
            assert rs[0][0] == 0 and rs[-1][1] == T and all(a[1] == b[0] for a, b in zip(rs, rs[1:]))
            assert all((b - a) % 512 == 0 for a, b in rs[:-1] if b < T)


def test_file_descriptors_cross_a_socket():
    # the exported handle of a slice is a POSIX file descriptor; peers receive it over a Unix socket
    import os
    import socket
    from paper_2608_07524_b200 import vmm
    a, b = socket.socketpair(socket.AF_UNIX, socket.SOCK_STREAM)
    r1, w1 = os.pipe()
    r2, w2 = os.pipe()
    vmm.send_fds(a, [w1, w2])
    got = vmm.recv_fds(b, 2)
    assert len(got) == 2 and got[0] not in (w1, w2)
    os.write(got[0], b"one")
    os.write(got[1], b"two")
    assert os.read(r1, 3) == b"one" and os.read(r2, 3) == b"two"
    for fd in (r1, w1, r2, w2, *got):
        os.close(fd)
    a.close()
    b.close()


def test_head_groups():
    from paper_2608_07524_b200.seqpar import head_group
    assert [head_group(r, 4, 16) for r in range(4)] == [slice(0, 4), slice(4, 8), slice(8, 12), slice(12, 16)]
    with pytest.raises(ValueError):
        head_group(0, 3, 16)


@pytest.mark.gpu
def test_attention_in_place_on_mapped_token_shards():
    """Three virtual ranks on one GPU: q, k, v, o, dO, dq, dk, dv are [T, H, d] ranges stitched from three
    separate physical allocations each (the single-GPU stand-in for slices that live on three GPUs); every
    virtual rank runs its head group in place on them; the result must match the oracle, and the plain
    kernels on ordinary tensors bit for bit (dq within rounding)."""
    import numpy as np
    import oracle
    from paper_2608_07524_b200 import binding as B
    from paper_2608_07524_b200 import inputs, vmm
    from paper_2608_07524_b200.seqpar import sp_attention_bwd_mapped, sp_attention_fwd_mapped
    dev, p, H, d = 0, 3, 12, 128           # 3072 bytes per token: 2048 tokens per 6 MB (three granules)
    lengths = [1500, 700, 129, 64, 2500, 13, 300]          # 5206 tokens: sequences straddle the slice boundaries
    T = sum(lengths)
    cu = np.concatenate([[0], np.cumsum(lengths)]).astype(np.int32)
    tensors, ranges, keep = vmm.stitched_tensors_local(T, H, d, p, dev, 8)
    assert ranges == [(0, 2048), (2048, 4096), (4096, T)] and len(keep[0].slices) == 3
    q, k, v, o, g, dq, dk, dv = tensors
    src = inputs.make_qkvg(T, H, d, 98)
    for dst, x in zip((q, k, v, g), src):
        dst.copy_(x)
    for out in (o, dq, dk, dv):
        out.fill_(float("nan"))
    cud = torch.tensor(cu, device="cuda")
    lses = [sp_attention_fwd_mapped(q, k, v, o, cud, max(lengths), True, r, p) for r in range(p)]
    for r in range(p):
        sp_attention_bwd_mapped(q, k, v, o, g, lses[r], dq, dk, dv, cud, max(lengths), True, r, p)
    torch.cuda.synchronize()
    qc, kc, vc, gc = (x.cuda() for x in src)
    ref_o, ref_lse = B.dcp_varlen_attn_fwd(qc, kc, vc, cud, max(lengths), True)
    ref = B.dcp_varlen_attn_bwd(qc, kc, vc, ref_o, gc, ref_lse, cud, max(lengths), True)
    assert torch.equal(o, ref_o) and torch.equal(torch.cat(lses, 0), ref_lse)
    assert torch.equal(dk, ref[1]) and torch.equal(dv, ref[2])
    assert float((dq.float() - ref[0].float()).abs().max()) <= 2e-2
    O, L = oracle.attn_fwd(*src[:3], cu, True)
    rdq, rdk, rdv = oracle.attn_bwd(*src, cu, True)
    for name, got, want in (("o", o, O), ("dq", dq, rdq), ("dk", dk, rdk), ("dv", dv, rdv)):
        got = got.double().cpu().numpy()
        assert float(np.max(np.abs(got - want))) <= 5e-2 and float(np.linalg.norm(got - want) / np.linalg.norm(want)) <= 1e-2, name
    del tensors, q, k, v, o, g, dq, dk, dv
    for rng in keep:
        rng.close()


def _fd_worker(rank, p, socket_dir, out):
    import os
    from paper_2608_07524_b200 import vmm
    pipes = [os.pipe() for _ in range(2)]                       # stand-ins for two exported allocations
    got = vmm.exchange_fds(rank, p, [w for _, w in pipes], socket_dir, "t")
    for peer in range(p):
        if peer != rank:
            for t, fd in enumerate(got[peer]):
                os.write(fd, bytes([10 * rank + t]))            # "rank `rank` was here", through the PEER's pipe
                os.close(fd)
    # every peer has written one byte into each of my pipes
    seen = [sorted(os.read(r, 1)[0] for _ in range(p - 1)) for r, _ in pipes]
    out.put((rank, got[rank] is None, seen))


def test_descriptor_exchange_between_three_processes(tmp_path):
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    p = 3
    procs = [ctx.Process(target=_fd_worker, args=(r, p, str(tmp_path), out)) for r in range(p)]
    for pr in procs:
        pr.start()
    results = sorted(out.get(timeout=120) for _ in range(p))
    for pr in procs:
        pr.join(timeout=60)
        assert pr.exitcode == 0
    for rank, own_is_none, seen in results:
        others = [r for r in range(p) if r != rank]
        assert own_is_none and seen == [[10 * r for r in others], [10 * r + 1 for r in others]]


def _owner_process(sock, nbytes, seed):
    # a second process on the same GPU: owns a slice, fills it, exports it, hands the descriptor over
    import torch as th
    from paper_2608_07524_b200 import vmm
    th.zeros(1, device="cuda:0")
    s = vmm.Slice(nbytes, 0)
    rng = vmm.StitchedRange([s], 0)
    t = rng.tensor((nbytes // 2,), th.bfloat16)
    g = th.Generator(device="cuda").manual_seed(seed)
    t.copy_(th.randn(nbytes // 2, generator=g, device="cuda").to(th.bfloat16))
    th.cuda.synchronize()
    sock.settimeout(120)                                      # never outlive a failed parent
    vmm.send_fds(sock, [s.export_fd()])
    assert sock.recv(1) == b"k"                               # the peer has read what it wanted
    del t
    rng.close()
    s.release()


@pytest.mark.gpu
def test_a_slice_owned_by_another_process_is_mapped_and_read():
    """The descriptor path between processes, on one GPU: a child process creates and fills a slice and
    exports it; this process imports it, maps it behind a slice of its own, and reads both through one range."""
    from paper_2608_07524_b200 import vmm
    torch.zeros(1, device="cuda:0")
    gran = vmm.granularity(0)
    a, b = socket.socketpair(socket.AF_UNIX, socket.SOCK_STREAM)
    ctx = mp.get_context("spawn")
    child = ctx.Process(target=_owner_process, args=(b, gran, 123), daemon=True)
    child.start()
    b.close()
    a.settimeout(120)
    try:
        (fd,) = vmm.recv_fds(a, 1)
        mine = vmm.Slice(gran, 0)
        theirs = vmm.Slice.import_fd(fd, gran, 0)
        os.close(fd)
        rng = vmm.StitchedRange([mine, theirs], 0)
        t = rng.tensor((gran,), torch.bfloat16)                    # 2 granules of bf16
        t[: gran // 2].fill_(3.0)
        g = torch.Generator(device="cuda").manual_seed(123)
        want = torch.randn(gran // 2, generator=g, device="cuda").to(torch.bfloat16)
        same = torch.equal(t[gran // 2:], want) and bool((t[: gran // 2] == 3.0).all())
        a.sendall(b"k")
    finally:
        a.close()                                                  # a waiting child sees end-of-file and leaves
    child.join(timeout=60)
    assert same and child.exitcode == 0
    del t
    rng.close()
    mine.release()
    theirs.release()
