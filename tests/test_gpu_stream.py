"""The end-to-end stream on real data: a batch is planned, its sequences are gathered into the
micro-batches the plan names, every micro-batch runs forward (+ a recompute forward) + backward, and
the results are scattered back to the batch's order.  Outputs are compared with the fp64 oracle run on
the UNSPLIT batch (attention is per sequence, so splitting must not change anything) and the plan with
the brute-force planner oracle.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2608_07524_b200 import binding as B
from paper_2608_07524_b200 import inputs
from paper_2608_07524_b200.profiler import intra_candidates, select_group_setting
from paper_2608_07524_b200.stream import StreamRunner, plan_batch, plan_length_group

pytestmark = pytest.mark.gpu

MAX_ABS, REL_FRO, LSE_ABS = 5e-2, 1e-2, 2e-3
LENGTHS = [130, 13, 1200, 13, 64, 64, 13, 100, 600, 300, 256, 1200, 300, 1200, 64, 130, 13, 16, 1200, 300]
H, D, LAYERS, T_C, BUDGET = 2, 64, 2, 1 << 20, 1587987       # binds: four micro-batches, three of them recompute


def close(name, got, ref):
    got = got.detach().double().cpu().numpy()
    assert np.all(np.isfinite(got)), name
    max_abs = float(np.max(np.abs(got - ref)))
    rel = float(np.linalg.norm(got - ref) / max(np.linalg.norm(ref), 1e-30))
    assert max_abs <= MAX_ABS and rel <= REL_FRO, f"{name}: max-abs {max_abs:.3e}, rel-Frobenius {rel:.3e}"


def load_batch(runner, q, k, v, g):
    T = q.shape[0]
    for dst, src in ((runner.q, q), (runner.k, k), (runner.v, v), (runner.g, g)):
        dst[:T].copy_(src)
    for out in (runner.o, runner.dq, runner.dk, runner.dv):
        out.fill_(float("nan"))
    runner.lse.fill_(float("nan"))


@pytest.mark.parametrize("causal", [False, True])
def test_planned_stream_matches_the_oracle_on_the_unsplit_batch(causal):
    T = sum(LENGTHS)
    cu = np.concatenate([[0], np.cumsum(LENGTHS)]).astype(np.int32)
    q, k, v, g = inputs.make_qkvg(T, H, D, 70)
    plan = plan_batch(LENGTHS, BUDGET, H, D, n_layers=LAYERS, fixed_cost=T_C)
    # the plan itself, bit for bit against the enumeration of every split
    assert (plan.mb_id, plan.recompute, plan.cost) == oracle.plan_bruteforce(LENGTHS, BUDGET, n_heads=H, head_dim=D,
                                                                             n_layers=LAYERS, fixed_cost=T_C)
    K = len(plan.recompute)
    assert K >= 2 and max(plan.recompute) >= 1 and min(plan.recompute) == 0
    # micro-batch k holds exactly the sequences the planner put there, in input order
    for kk, mb in enumerate(plan.micro_batches):
        members = [i for i in range(len(LENGTHS)) if plan.mb_id[i] == kk]
        assert list(mb.seq_index) == members and list(mb.lengths) == [LENGTHS[i] for i in members]
        assert int(mb.seg[:, 2].sum()) == sum(LENGTHS[i] for i in members)

    runner = StreamRunner(T, len(LENGTHS), H, D, causal, "cuda")
    runner.verify_recompute = True
    load_batch(runner, q, k, v, g)
    assert runner.run_batch(plan, T) == T
    runner.check()
    assert runner.recompute_mismatches == 0          # the re-run forward reproduces o and lse bit for bit
    split = [x[:T].clone() for x in (runner.o, runner.dq, runner.dk, runner.dv)] + [runner.lse[: H * T].view(H, T).clone()]

    O, L = oracle.attn_fwd(q, k, v, cu, causal)
    rdq, rdk, rdv = oracle.attn_bwd(q, k, v, g, cu, causal)
    close("o", split[0], O)
    close("dq", split[1], rdq)
    close("dk", split[2], rdk)
    close("dv", split[3], rdv)
    assert float(np.max(np.abs(split[4].double().cpu().numpy() - L))) <= LSE_ABS

    # the same batch under a budget that does not bind runs in place as one micro-batch: per-sequence
    # results are the same kernels on the same rows, whatever else shares the launch
    whole = plan_batch(LENGTHS, 10 ** 12, H, D, n_layers=LAYERS, fixed_cost=T_C)
    assert len(whole.micro_batches) == 1 and whole.micro_batches[0].seg is None
    load_batch(runner, q, k, v, g)
    runner.run_batch(whole, T)
    runner.check()
    # sequences longer than a tile run the same instructions on the same data either way: bit-identical (dq
    # is summed by atomics in arbitrary order).  Shorter ones share tiles with whatever neighbours they have,
    # which moves them to other rows of the tile and changes the order of some fp32 sums: within rounding.
    long_rows = torch.from_numpy(np.concatenate([np.arange(cu[b], cu[b + 1]) for b, L in enumerate(LENGTHS) if L > 128])).cuda()
    whole_out = (runner.o[:T], runner.dq[:T], runner.dk[:T], runner.dv[:T])
    for i in (0, 2, 3):
        assert torch.equal(whole_out[i][long_rows], split[i][long_rows])
    assert torch.equal(runner.lse[: H * T].view(H, T)[:, long_rows], split[4][:, long_rows])
    for i in range(4):
        assert float((whole_out[i].float() - split[i].float()).abs().max()) <= 2e-2
    assert float((runner.lse[: H * T].view(H, T) - split[4]).abs().max()) <= 1e-4


def test_copy_segments_gathers_and_scatters():
    dev = "cuda"
    rng = np.random.default_rng(12)
    lengths = [int(x) for x in rng.integers(0, 300, size=40)]
    mb_id = [int(x) for x in rng.integers(0, 3, size=40)]
    T = sum(lengths)
    src_cu = np.concatenate([[0], np.cumsum(lengths)])
    offs, index, mb_cu, seg_off, seg = B.dcp_plan_segments(lengths, mb_id, 3, 50)
    x = torch.randn((T, 3, 8), device=dev).to(torch.bfloat16)
    lse = torch.randn((5, T), device=dev)
    back = torch.zeros_like(x)
    lse_back = torch.zeros_like(lse)
    for k in range(3):
        members = index[offs[k]: offs[k + 1]]
        Tk = sum(lengths[i] for i in members)
        segk = torch.tensor(seg[seg_off[k]: seg_off[k + 1]], dtype=torch.int32, device=dev).contiguous()
        got = torch.full((Tk + 4, 3, 8), 7.0, dtype=torch.bfloat16, device=dev)
        B.dcp_copy_segments(x, got, segk, segk.shape[0], 3 * 8 * 2)
        want = torch.cat([x[src_cu[i]: src_cu[i + 1]] for i in members] + [x[:0]])
        assert torch.equal(got[:Tk], want) and bool((got[Tk:] == 7.0).all())
        # 4-byte rows in planes (the layout of lse), gather then scatter
        lk = torch.zeros((5, Tk), device=dev)
        B.dcp_copy_segments(lse, lk, segk, segk.shape[0], 4, n_planes=5, src_plane_bytes=4 * T, dst_plane_bytes=4 * Tk)
        assert torch.equal(lk, torch.cat([lse[:, src_cu[i]: src_cu[i + 1]] for i in members] + [lse[:, :0]], dim=1))
        B.dcp_copy_segments(got, back, segk, segk.shape[0], 3 * 8 * 2, reverse=True)
        B.dcp_copy_segments(lk, lse_back, segk, segk.shape[0], 4, reverse=True, n_planes=5, src_plane_bytes=4 * Tk,
                            dst_plane_bytes=4 * T)
    assert torch.equal(back, x) and torch.equal(lse_back, lse)


def test_algorithm_1_setting_measured_on_the_device_and_applied():
    """DCP-intra on one GPU (p = 1): the candidate table (b, 1) for one sequence length is measured the
    dual-layer way on this device, Algorithm 1 selects batch size and recompute count under a memory
    capacity, the selection is compared with the exhaustive oracle on the SAME measured table, and a group
    of sequences of that length is then run with the selected setting and compared with the attention
    oracle."""
    L, n_seqs, lam = 384, 7, 4
    cands = intra_candidates(L, [1, 2, 4], H, D, False, lam, fixed_cost_ns=20000)
    assert all(c[2] > 0 and c[4] > lam * 2 * c[2] for c in cands)
    unit = L * H * D * 2
    # room for b = 4 with nothing kept, for b = 2 with two layers kept, for b = 1 with all four kept
    capacity = lam * 4 * unit + 4 * unit
    b, r, t = select_group_setting(cands, capacity, lam)
    idx, r_ref, t_ref = oracle.intra_select(cands, capacity, lam)
    assert (b, r, t) == (cands[idx][0], r_ref, t_ref)
    if r == 0:                                     # make sure the recompute path runs whatever the device measured
        capacity = lam * b * unit + b * unit * 4 * (lam - 1)
        b2, r, t = select_group_setting([c for c in cands if c[0] == b], capacity, lam)
        assert b2 == b and r == 1
    plan = plan_length_group(n_seqs, L, b, r)
    assert len(plan.micro_batches) == -(-n_seqs // b) and all(m.recompute == r for m in plan.micro_batches)
    T = n_seqs * L
    cu = np.arange(0, T + 1, L, dtype=np.int32)
    q, k, v, g = inputs.make_qkvg(T, H, D, 71)
    runner = StreamRunner(T, n_seqs, H, D, False, "cuda")
    runner.verify_recompute = True
    load_batch(runner, q, k, v, g)
    assert runner.run_batch(plan, T) == T
    runner.check()
    assert runner.recompute_mismatches == 0
    O, Lse = oracle.attn_fwd(q, k, v, cu, False)
    rdq, rdk, rdv = oracle.attn_bwd(q, k, v, g, cu, False)
    close("o", runner.o[:T], O)
    close("dq", runner.dq[:T], rdq)
    close("dk", runner.dk[:T], rdk)
    close("dv", runner.dv[:T], rdv)
    assert float(np.max(np.abs(runner.lse[: H * T].view(H, T).double().cpu().numpy() - Lse))) <= LSE_ABS


def test_algorithm_1_candidates_over_batch_size_and_sequence_parallel_size():
    """Algorithm 1's table with both of its dimensions: rows (b, p) for p = 1, 2, 4, each measured on this device
    as one rank's share (its heads of all tokens, in place inside full-width tensors; what crosses NVLink is
    not in a one-GPU measurement).  The selection is compared with the exhaustive oracle on the SAME table, with
    room for everything and with so little memory that only a sharded setting fits."""
    L, heads, lam = 8192, 16, 4                       # enough work that a quarter of the heads takes visibly less time
    cands = intra_candidates(L, [1, 2], heads, 128, False, lam, fixed_cost_ns=20000, sp_sizes=(1, 2, 4))
    assert [(c[0], c[1]) for c in cands] == [(1, 1), (2, 1), (1, 2), (2, 2), (1, 4), (2, 4)]
    assert all(c[2] > 0 and c[4] > 0 for c in cands)
    by = {(c[0], c[1]): c for c in cands}
    for b in (1, 2):                                   # a rank of a larger group holds less and works less
        assert by[(b, 1)][5] > by[(b, 2)][5] > by[(b, 4)][5]
        assert by[(b, 1)][2] > by[(b, 4)][2]
    roomy = 1 << 40
    idx, r, t = B.dcp_intra_select(cands, roomy, lam)
    assert (idx, r, t) == oracle.intra_select(cands, roomy, lam) and r == 0
    # less than any p = 1 row needs even with every layer recomputed; (1, 2), (1, 4) and (2, 4) still fit
    tight = min(by[(1, 1)][5], by[(2, 1)][5]) - 1
    assert tight >= by[(1, 2)][5] and tight >= by[(2, 4)][5]
    idx, r, t = B.dcp_intra_select(cands, tight, lam)
    assert (idx, r, t) == oracle.intra_select(cands, tight, lam) and cands[idx][1] >= 2
