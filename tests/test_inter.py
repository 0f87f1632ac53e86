"""DCP-inter step-count search (Section 3.3 Eq. 3, Appendix C): pins for the brute-force oracle and
bit-exact parity of the product's candidate-makespan search against it."""
import numpy as np
import pytest

import oracle
from paper_2608_07524_b200 import binding as B
from paper_2608_07524_b200 import inputs


def idle_of(T, g):
    m = max(gi * ti for gi, ti in zip(g, T))
    return sum(m - gi * ti for gi, ti in zip(g, T))


# ---------------------------------------------------------------- oracle pins
def test_oracle_hand_worked_cases():
    # T = (2, 3), G_max = 2: iterations up to 6 allowed; g = (3, 2) gives 6 = 6, no idle time
    assert oracle.inter_bruteforce([2, 3], 1, 2) == ([3, 2], 0)
    # G_max = 1: only g = (1, 1) fits under the 3-unit cap; idle = 3 - 2
    assert oracle.inter_bruteforce([2, 3], 1, 1) == ([1, 1], 1)
    # T = (10, 11), G_max = 4 (cap 44): candidates leave idle >= 1; (1, 1) is the shortest with idle 1
    assert oracle.inter_bruteforce([10, 11], 1, 4) == ([1, 1], 1)
    # G_max = 10 reaches the common multiple 110
    assert oracle.inter_bruteforce([10, 11], 1, 10) == ([11, 10], 0)
    # equal batches: one step each, then G_min = 3 scales every count by 3 (idle stays 0)
    assert oracle.inter_bruteforce([7, 7, 7], 3, 4) == ([3, 3, 3], 0)
    # multiples of the fastest batch balance exactly: g_i = T_max / T_i
    assert oracle.inter_bruteforce([1, 2, 4, 8], 1, 1) == ([8, 4, 2, 1], 0)
    # G_min scaling multiplies idle too: best is (1, 1) with idle 1, scaled by ceil(5 / 1)
    assert oracle.inter_bruteforce([10, 11], 5, 4) == ([5, 5], 5)


def test_oracle_invariants():
    rng = np.random.default_rng(0)
    for _ in range(200):
        n = int(rng.integers(1, 5))
        T = [int(x) for x in rng.integers(1, 40, size=n)]
        g_max = int(rng.integers(1, 5))
        g, idle = oracle.inter_bruteforce(T, 1, g_max)
        assert all(x >= 1 for x in g) and idle == idle_of(T, g) and idle >= 0
        assert max(gi * ti for gi, ti in zip(g, T)) <= g_max * max(T)
        assert idle <= idle_of(T, [1] * n)                       # never worse than no accumulation
        # scaling every time by a constant keeps g and scales the idle time
        g2, idle2 = oracle.inter_bruteforce([3 * t for t in T], 1, g_max)
        assert g2 == g and idle2 == 3 * idle
        # more head-room never hurts
        _, idle3 = oracle.inter_bruteforce(T, 1, g_max + 1)
        assert idle3 <= idle
        # permuting the batches permutes... the optimum value (the vector may differ only by the tie rule)
        perm = rng.permutation(n)
        _, idle4 = oracle.inter_bruteforce([T[i] for i in perm], 1, g_max)
        assert idle4 == idle


# ---------------------------------------------------------------- product vs oracle
def test_product_matches_bruteforce():
    rng = np.random.default_rng(1)
    for _ in range(1500):
        n = int(rng.integers(1, 6))
        T = [int(x) for x in rng.integers(1, 60, size=n)]
        g_max = int(rng.integers(1, 6))
        g_min = int(rng.integers(1, 8))
        try:
            ref = oracle.inter_bruteforce(T, g_min, g_max)
        except ValueError:
            continue
        g, idle, it = B.dcp_inter_plan(T, g_min, g_max)
        assert (g, idle) == ref, (T, g_min, g_max)
        assert it == max(gi * ti for gi, ti in zip(g, T))


def test_product_on_modelled_stream_batches():
    """Eight virtual workers, one config-5 batch each, times from the planner's model (7 * sum L^2):
    accumulation steps cut the idle fraction the paper calls the imbalance ratio (Section 4.2)."""
    batches = inputs.stream_batches()[:8]
    T = [7 * sum(L * L for L in b) // 10 ** 6 for b in batches]
    g, idle, it = B.dcp_inter_plan(T, 1, 4)
    ratio = idle / (len(T) * it)
    ratio_plain = idle_of(T, [1] * 8) / (8 * max(T))
    assert ratio <= ratio_plain and ratio < 0.25
    assert max(gi * ti for gi, ti in zip(g, T)) <= 4 * max(T)


def test_errors():
    for bad in ([], [0, 3], [-1]):
        with pytest.raises(B.DcpError) as e:
            B.dcp_inter_plan(bad)
        assert e.value.code == B.DCP_ERR_INVALID_ARG
    with pytest.raises(B.DcpError) as e:
        B.dcp_inter_plan([1, 2], g_min=0)
    assert e.value.code == B.DCP_ERR_INVALID_ARG
    # times whose ratio makes the candidate list explode are refused instead of searched for minutes
    with pytest.raises(B.DcpError) as e:
        B.dcp_inter_plan([1, 10 ** 9], 1, 4)
    assert e.value.code == B.DCP_ERR_UNSUPPORTED
    # int64-sized times are handled exactly
    g, idle, it = B.dcp_inter_plan([2 ** 61, 2 ** 61], 1, 2)
    assert g == [1, 1] and idle == 0 and it == 2 ** 61
