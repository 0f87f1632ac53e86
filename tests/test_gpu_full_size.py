"""Full-size benchmark configurations (2 text, 3 video, 4 extreme imbalance, and the video clips
seen along the spatial axis of a 2-D model) in the launch configuration the benchmark times; the
temporal axis (20384 sequences of 1-13 tokens) is small enough for the oracle to check in full.  A full fp64 evaluation of these is 10^13-10^14 flop, so the
oracle checks (a) every sequence of at most 8192 tokens completely, on every head, (b) for longer
sequences sampled query rows (O, lse, dQ) and key columns (dK, dV), which the definition lets it
compute one by one - at least 256 rows on every head of the longest sequence, key columns from its
first blocks included - plus one whole head of O and lse, and (c) two whole-tensor identities that
hold at any size:
    sum_i <Q_i, dQ_i> = sum_j <K_j, dK_j>      and      sum_j dV_j = sum_i dO_i
per (sequence, head), evaluated on the GPU results in fp64.  Their bounds have two parts: the
independent bf16 rounding of every stored gradient element (8 sigma), and a term proportional to
the absolute sum for the tensor cores' fp32 accumulation, which truncates instead of rounding and
so biases sums of thousands of partial products by about 1e-4 of their magnitude.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2608_07524_b200 import binding as B
from paper_2608_07524_b200 import inputs
from test_gpu_attn import Guarded

pytestmark = pytest.mark.gpu

MAX_ABS, REL_FRO, LSE_ABS = 5e-2, 1e-2, 2e-3
EPS_BF16 = 2.0 ** -9
ACC_BIAS = 5e-4


def close(name, got, ref):
    got = got.detach().double().cpu().numpy()
    max_abs = float(np.max(np.abs(got - ref)))
    rel = float(np.linalg.norm(got - ref) / max(np.linalg.norm(ref), 1e-30))
    assert np.all(np.isfinite(got)), name
    assert max_abs <= MAX_ABS and rel <= REL_FRO, f"{name}: max-abs {max_abs:.3e}, rel-Frobenius {rel:.3e}"


def sample_positions(L, rng, n_random=24):
    fixed = [0, 1, 127, 128, 255, 256, L - 257, L - 256, L - 129, L - 128, L - 2, L - 1, L // 2]
    pos = {p for p in fixed if 0 <= p < L}
    pos.update(int(x) for x in rng.integers(0, L, size=n_random))
    return np.array(sorted(pos), np.int32)


def workload_of(param, head_dim=128):
    if isinstance(param, int):
        return inputs.config(param)
    return inputs.Workload(param, inputs.short2d_lengths(param[:-2]), 16, head_dim, False, 12)


@pytest.fixture(scope="module", params=[2, 3, 4, "spatial2d"])
def full_run(request):
    w = workload_of(request.param)
    dev = "cuda"
    q, k, v, g = inputs.make_qkvg_device(w.total_tokens, w.n_heads, w.head_dim, w.value_seed, dev)
    cud = torch.tensor(w.cu_seqlens, dtype=torch.int32, device=dev)
    # outputs and workspace carry a poisoned margin after their end (a store past the last row shows there)
    buf = Guarded(w.total_tokens, w.n_heads, w.head_dim, len(w.lengths), dev)
    o, lse = B.dcp_varlen_attn_fwd(q, k, v, cud, w.max_seqlen, w.causal, out=buf.o, lse=buf.lse, workspace=buf.ws)
    B.dcp_query_status(buf.ws)
    buf.assert_margins_untouched("forward")
    dq, dk, dv = B.dcp_varlen_attn_bwd(q, k, v, o, g, lse, cud, w.max_seqlen, w.causal, dq=buf.dq, dk=buf.dk, dv=buf.dv,
                                       workspace=buf.ws)
    B.dcp_query_status(buf.ws)
    buf.assert_margins_untouched("backward")
    del buf.ws, buf.ws_raw
    host = tuple(x.cpu() for x in (q, k, v, g))
    yield w, (q, k, v, g), host, (o, lse, dq, dk, dv)
    torch.cuda.empty_cache()


FULL_LIMIT = 8192      # sequences up to this length are compared in full, on every head


def test_sequences_up_to_8192_tokens_in_full(full_run):
    """Every sequence of at most 8192 tokens, every head, every element of o, lse, dq, dk, dv.  The
    oracle sees them packed back to back as a batch of their own (attention is per sequence)."""
    w, _, (q, k, v, g), (o, lse, dq, dk, dv) = full_run
    seqs = [b for b, L in enumerate(w.lengths) if 0 < L <= FULL_LIMIT]
    if not seqs:
        pytest.skip("no sequence of at most 8192 tokens")
    rows = np.concatenate([np.arange(w.cu_seqlens[b], w.cu_seqlens[b + 1]) for b in seqs])
    sub_cu = np.concatenate([[0], np.cumsum([w.lengths[b] for b in seqs])]).astype(np.int32)
    idx_h = torch.from_numpy(rows)
    qs, ks, vs, gs = (x[idx_h].contiguous() for x in (q, k, v, g))
    O, Lse = oracle.attn_fwd(qs, ks, vs, sub_cu, w.causal)
    rdq, rdk, rdv = oracle.attn_bwd(qs, ks, vs, gs, sub_cu, w.causal)
    idx = idx_h.cuda()
    close("o", o[idx], O)
    close("dq", dq[idx], rdq)
    close("dk", dk[idx], rdk)
    close("dv", dv[idx], rdv)
    assert float(np.max(np.abs(lse[:, idx].double().cpu().numpy() - Lse))) <= LSE_ABS


def test_long_sequences_by_rows_columns_and_one_full_head(full_run):
    """Sequences longer than 8192 tokens.  The longest one: at least 256 sampled query rows (o, lse, dq) on
    EVERY head, one head's o and lse completely, and sampled key columns (dk, dv) that include the first key
    blocks - under a causal mask those are the columns that accumulate over the most query tiles (up to 1024
    for the 131072-token sequence), and the oracle needs the statistics of every later row for them, i.e.
    one full pass over the head.  The other long sequences: sampled rows on two heads and columns on one."""
    w, _, (q, k, v, g), (o, lse, dq, dk, dv) = full_run
    rng = np.random.default_rng(100 + len(w.lengths))
    long_seqs = [b for b, L in enumerate(w.lengths) if L > FULL_LIMIT]
    if not long_seqs:
        pytest.skip("no sequence longer than 8192 tokens")
    longest = max(long_seqs, key=lambda b: w.lengths[b])
    for seq in long_seqs:
        L, c0 = w.lengths[seq], w.cu_seqlens[seq]
        heads = range(w.n_heads) if seq == longest else (0, w.n_heads - 1)
        for head in heads:
            rows = sample_positions(L, rng, n_random=260 if seq == longest else 24)
            assert seq != longest or rows.size >= 256
            Or, lr, dqr = oracle.attn_rows(q, k, v, g, w.cu_seqlens, w.causal, seq, head, rows)
            idx = torch.tensor(c0 + rows, device="cuda").long()
            close(f"o seq {seq} head {head}", o[idx, head], Or)
            close(f"dq seq {seq} head {head}", dq[idx, head], dqr)
            assert float(np.max(np.abs(lse[head, idx].double().cpu().numpy() - lr))) <= LSE_ABS
        head = 1
        cols = sample_positions(L, rng, n_random=8)
        if seq == longest:
            early = np.concatenate([[0, 1, 127, 128, 255], rng.integers(0, 4096, size=8)])
            cols = np.unique(np.concatenate([cols, early])).astype(np.int32)
        elif w.causal:
            cols = cols[cols >= L - 2048]          # keeps the row pass short for the sequences that are not the longest
        dkc, dvc = oracle.attn_cols(q, k, v, g, w.cu_seqlens, w.causal, seq, head, cols)
        idx = torch.tensor(c0 + cols, device="cuda").long()
        close(f"dk seq {seq}", dk[idx, head], dkc)
        close(f"dv seq {seq}", dv[idx, head], dvc)
    # one whole head of the longest sequence
    L, c0, head = w.lengths[longest], w.cu_seqlens[longest], 2
    sl = slice(c0, c0 + L)
    O, Lse = oracle.attn_fwd(q[sl, head:head + 1].contiguous(), k[sl, head:head + 1].contiguous(),
                             v[sl, head:head + 1].contiguous(), [0, L], w.causal)
    close("o, one full head", o[sl, head:head + 1], O)
    assert float(np.max(np.abs(lse[head:head + 1, sl].double().cpu().numpy() - Lse))) <= LSE_ABS


def test_whole_tensor_identities(full_run):
    w, (q, k, v, g), _, (o, lse, dq, dk, dv) = full_run
    for seq, L in enumerate(w.lengths):
        sl = slice(w.cu_seqlens[seq], w.cu_seqlens[seq] + L)
        qd = q[sl].double() * dq[sl].double()
        kd = k[sl].double() * dk[sl].double()
        lhs, rhs = qd.sum(dim=(0, 2)), kd.sum(dim=(0, 2))
        # both sides carry independent bf16 rounding of every gradient element
        bound = (8 * EPS_BF16 * torch.sqrt((qd * qd).sum(dim=(0, 2)) + (kd * kd).sum(dim=(0, 2)))
                 + ACC_BIAS * (qd.abs().sum(dim=(0, 2)) + kd.abs().sum(dim=(0, 2))) + 1e-6)
        assert bool(((lhs - rhs).abs() <= bound).all()), f"<Q,dQ> vs <K,dK> on sequence {seq}"
        del qd, kd
        dvs = dv[sl].double()
        lhs, rhs = dvs.sum(dim=0), g[sl].double().sum(dim=0)
        bound = 8 * EPS_BF16 * torch.sqrt((dvs * dvs).sum(dim=0)) + ACC_BIAS * dvs.abs().sum(dim=0) + 1e-6
        assert bool(((lhs - rhs).abs() <= bound).all()), f"sum dV vs sum dO on sequence {seq}"
    assert bool(torch.isfinite(o.float()).all()) and bool(torch.isfinite(lse).all())


@pytest.mark.parametrize("head_dim", [128, 72])
def test_temporal_axis_in_full(head_dim):
    """Thousands of 1-13 token sequences, merged by the work-list kernels into tiles of up to 128
    tokens: every output element against the oracle.  72 is the head dimension of the paper's
    second model (it runs zero-padded to 128 columns)."""
    w = workload_of("temporal2d", head_dim)
    q, k, v, g = inputs.make_qkvg_device(w.total_tokens, w.n_heads, w.head_dim, w.value_seed, "cuda")
    cud = torch.tensor(w.cu_seqlens, dtype=torch.int32, device="cuda")
    ws = B.alloc_workspace(w.total_tokens, len(w.lengths), w.n_heads, w.head_dim, True, "cuda")
    o, lse = B.dcp_varlen_attn_fwd(q, k, v, cud, w.max_seqlen, w.causal, workspace=ws)
    dq, dk, dv = B.dcp_varlen_attn_bwd(q, k, v, o, g, lse, cud, w.max_seqlen, w.causal, workspace=ws)
    B.dcp_query_status(ws)
    qc, kc, vc, gc = (x.cpu() for x in (q, k, v, g))
    O, Lse = oracle.attn_fwd(qc, kc, vc, w.cu_seqlens, w.causal)
    rdq, rdk, rdv = oracle.attn_bwd(qc, kc, vc, gc, w.cu_seqlens, w.causal)
    close("o", o, O)
    close("dq", dq, rdq)
    close("dk", dk, rdk)
    close("dv", dv, rdv)
    assert float(np.max(np.abs(lse.double().cpu().numpy() - Lse))) <= LSE_ABS


@pytest.mark.parametrize("cfg", [2, 3])
def test_full_size_outputs_do_not_depend_on_neighbours(cfg):
    """Replace one sequence's q, k, v, dO (the second longest) and run again: every other sequence's o,
    lse, dk and dv must come out bit for bit the same (dq is summed by atomics in arbitrary order once
    a sequence has more than two key blocks, so it is compared within rounding)."""
    w = inputs.config(cfg)
    dev = "cuda"
    q, k, v, g = inputs.make_qkvg_device(w.total_tokens, w.n_heads, w.head_dim, w.value_seed, dev)
    cud = torch.tensor(w.cu_seqlens, dtype=torch.int32, device=dev)
    ws = B.alloc_workspace(w.total_tokens, len(w.lengths), w.n_heads, w.head_dim, True, dev)

    def run():
        o, lse = B.dcp_varlen_attn_fwd(q, k, v, cud, w.max_seqlen, w.causal, workspace=ws)
        dq, dk, dv = B.dcp_varlen_attn_bwd(q, k, v, o, g, lse, cud, w.max_seqlen, w.causal, workspace=ws)
        B.dcp_query_status(ws)
        return o, lse, dq, dk, dv

    a = run()
    victim = int(np.argsort(w.lengths)[-2])
    lo, hi = w.cu_seqlens[victim], w.cu_seqlens[victim + 1]
    gen = torch.Generator(device=dev).manual_seed(99)
    for x in (q, k, v, g):
        x[lo:hi] = (torch.randn(x[lo:hi].shape, generator=gen, device=dev) * 2).to(torch.bfloat16)
    b = run()
    keep = torch.ones(w.total_tokens, dtype=torch.bool, device=dev)
    keep[lo:hi] = False
    for i in (0, 3, 4):
        assert torch.equal(a[i][keep], b[i][keep])
    assert torch.equal(a[1][:, keep], b[1][:, keep])
    assert float((a[2][keep].float() - b[2][keep].float()).abs().max()) <= 3e-2
    assert not torch.equal(a[0][lo:hi], b[0][lo:hi])
