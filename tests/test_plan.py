"""The product planner (host C++, through the C ABI) must match the brute-force oracle bit-exactly:
micro-batch ids, recompute counts and cost."""
import os

import numpy as np
import pytest

import oracle
from paper_2608_07524_b200 import binding as B
from paper_2608_07524_b200 import inputs
from paper_2608_07524_b200.stream import plan_batch

GOLD = os.path.join(os.path.dirname(__file__), "golden", "plan_config1.txt")


def both(lengths, budget, **kw):
    try:
        ref = oracle.plan_bruteforce(lengths, budget, **kw)
    except oracle.Infeasible:
        ref = None
    try:
        got = B.dcp_plan(lengths, budget, **kw)
    except B.DcpError as e:
        assert e.code == B.DCP_ERR_INFEASIBLE
        got = None
    return got, ref


def test_config1_budget_sweep_matches_golden_and_oracle():
    with open(GOLD) as f:
        rows = [l.split() for l in f if l.strip() and not l.startswith("#")]
    for bud, lam, K, sizes, rec, cost in rows:
        kw = dict(n_heads=2, head_dim=64, n_layers=int(lam))
        got, ref = both([17, 64, 100, 255], int(bud), **kw)
        assert got == ref
        if K == "-":
            assert got is None
        else:
            assert got[1] == [int(x) for x in rec.split(",")] and got[2] == int(cost)


def test_random_cases_match_bruteforce():
    rng = np.random.default_rng(0)
    for _ in range(4000):
        n = int(rng.integers(1, 11))
        lengths = [int(x) for x in rng.integers(1, 500, size=n)]
        lam = int(rng.choice([1, 2, 4, 28]))
        TC = int(rng.choice([0, 1, 50, 10 ** 5, 1 << 24, 1 << 40]))
        unit = 2 * 8 * 2
        budget = int(rng.integers(max(lam * unit * max(lengths) - 40, 0), 5 * lam * unit * sum(lengths) + 2))
        got, ref = both(lengths, budget, n_heads=2, head_dim=8, n_layers=lam, fixed_cost=TC)
        assert got == ref, (lengths, budget, lam, TC)


def test_equal_lengths_and_ties():
    for n in range(1, 9):
        for budget in (100, 1000, 16 * 20 * 5, 16 * 20 * 5 + 1, 10 ** 6):
            got, ref = both([10] * n, budget, n_heads=1, head_dim=8, n_layers=1, fixed_cost=0)
            assert got == ref


def test_stream_batches_literal_and_binding_settings():
    batches = inputs.stream_batches()
    # literal config: Lambda = 1, 180 GB: nothing binds, one micro-batch without recompute
    for lengths in batches[:6]:
        got, ref = both(lengths, 180 * 10 ** 9)
        assert got == ref and got[1] == [0] and set(got[0]) == {0}
    # binding variant: 28 layers (the paper's Transformer-2D depth, Appendix B) under the paper's
    # 80 GB cap (Section 4.1): heavy batches split
    n_split = 0
    for lengths in batches[:6] + [max(batches, key=sum)]:
        got, ref = both(lengths, 80 * 10 ** 9, n_layers=28)
        assert got == ref
        n_split += len(got[1]) > 1
    assert n_split >= 1


def test_plan_batch_groups_sequences():
    lengths = [17, 64, 100, 255]
    plan = plan_batch(lengths, 65280, n_heads=2, head_dim=64)
    mbs = plan.micro_batches
    # micro-batch 0 holds the longest sequence; inside a micro-batch sequences keep their input order
    assert [list(m.lengths) for m in mbs] == [[255], [17, 64, 100]] and [m.recompute for m in mbs] == [1, 1]
    assert [list(m.seq_index) for m in mbs] == [[3], [0, 1, 2]] and plan.mb_id == [1, 1, 1, 0]
    # copy lists: (row in the batch, row in the micro-batch, rows), long sequences cut into pieces of 64 rows
    assert mbs[0].seg.tolist() == [[181, 0, 64], [245, 64, 64], [309, 128, 64], [373, 192, 63]]
    assert mbs[1].seg.tolist() == [[0, 0, 17], [17, 17, 64], [81, 81, 64], [145, 145, 36]]
    # a plan that does not split runs in place
    one = plan_batch(lengths, 10 ** 6, n_heads=2, head_dim=64)
    assert len(one.micro_batches) == 1 and one.micro_batches[0].seg is None
    assert list(one.micro_batches[0].lengths) == lengths


def reference_segments(lengths, mb_id, K, max_rows):
    """The layout written out plainly: per micro-batch the input indices in input order, its boundary
    array, and one copy piece per max_rows rows of every sequence."""
    src = np.concatenate([[0], np.cumsum(lengths)])
    offs, index, cu, seg_off, seg = [0], [], [], [0], []
    for k in range(K):
        members = [i for i in range(len(lengths)) if mb_id[i] == k]
        index += members
        offs.append(len(index))
        dst = 0
        cu.append(0)
        for i in members:
            for done in range(0, lengths[i], max_rows):
                seg.append([int(src[i]) + done, dst + done, min(max_rows, lengths[i] - done)])
            dst += lengths[i]
            cu.append(dst)
        seg_off.append(len(seg))
    return offs, index, cu, seg_off, seg


def test_plan_segments_against_a_plain_restatement():
    rng = np.random.default_rng(8)
    for _ in range(300):
        n = int(rng.integers(1, 30))
        lengths = [int(x) for x in rng.choice([0, 1, 5, 63, 64, 65, 128, 300, 1000], size=n)]
        K = int(rng.integers(1, n + 1))
        mb_id = [int(x) for x in rng.integers(0, K, size=n)]
        max_rows = int(rng.choice([1, 7, 64, 1000]))
        got = B.dcp_plan_segments(lengths, mb_id, K, max_rows)
        ref = reference_segments(lengths, mb_id, K, max_rows)
        assert [x.tolist() for x in got] == [list(x) for x in ref]
    with pytest.raises(B.DcpError) as e:
        B.dcp_plan_segments([5, 6], [0, 2], 2)
    assert e.value.code == B.DCP_ERR_INVALID_ARG


def test_errors():
    with pytest.raises(B.DcpError) as e:
        B.dcp_plan([5, 0], 1000)
    assert e.value.code == B.DCP_ERR_INVALID_ARG
    with pytest.raises(B.DcpError) as e:
        B.dcp_plan([], 1000)
    assert e.value.code == B.DCP_ERR_INVALID_ARG
    with pytest.raises(B.DcpError) as e:
        B.dcp_plan([5], -1)
    assert e.value.code == B.DCP_ERR_INVALID_ARG
    with pytest.raises(B.DcpError) as e:
        B.dcp_plan([5], 10, n_layers=0)
    assert e.value.code == B.DCP_ERR_INVALID_ARG
    with pytest.raises(B.DcpError) as e:      # cost beyond int64
        B.dcp_plan([2 ** 31 - 1] * 8, 2 ** 62, n_heads=1, head_dim=1, elt_bytes=1, n_layers=2 ** 31 - 1,
                   fixed_cost=2 ** 62)
    assert e.value.code in (B.DCP_ERR_OVERFLOW, B.DCP_ERR_INFEASIBLE)
    assert "dcp_plan" in B.lib().dcp_last_error().decode()
