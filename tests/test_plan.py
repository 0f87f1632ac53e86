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
    mbs = plan_batch(lengths, 65280, n_heads=2, head_dim=64)
    assert [m.lengths for m in mbs] == [[255], [100, 64, 17]] and [m.recompute for m in mbs] == [1, 1]


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
