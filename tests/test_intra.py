"""DCP-intra selection (Algorithm 1): the library's dcp_intra_select against the exhaustive oracle, and
the oracle against what Eq. 4-6 fix independently of any search: per candidate the number of layers
that may keep their activations has a closed form, and a hand-worked example."""
from fractions import Fraction

import numpy as np
import pytest

import oracle
from oracle.intra_oracle import Infeasible
from paper_2608_07524_b200 import binding as B


def from_closed_form(cands, M, L):
    """Eq. 6: M(r) = M_(b,p) + (L - r) m <= M  <=>  L - r <= (M - M_(b,p)) / m, so the smallest feasible r
    is L - min(L, floor((M - M_(b,p)) / m)); Eq. 5 then gives the time.  Best throughput over candidates."""
    best = None
    for idx, (b, p, t_f, m, T_bp, M_bp) in enumerate(cands):
        if M_bp > M:
            continue
        keep = L if m == 0 else min(L, (M - M_bp) // m)
        time = T_bp - keep * t_f
        key = (Fraction(b, p * time), -p, b, -idx)
        if best is None or key > best[0]:
            best = (key, idx, L - keep, time)
    return None if best is None else best[1:]


def random_case(rng):
    L = int(rng.integers(1, 30))
    n = int(rng.integers(1, 9))
    cands = []
    for _ in range(n):
        b, p = int(rng.integers(1, 9)), int(rng.choice([1, 2, 4, 8]))
        t_f = int(rng.integers(0, 1000))
        m = int(rng.integers(0, 500))
        T_bp = L * t_f + int(rng.integers(1, 5000))      # contains the recompute time of all L layers
        M_bp = int(rng.integers(0, 4000))
        cands.append((b, p, t_f, m, T_bp, M_bp))
    M = int(rng.integers(0, 6000))
    return cands, M, L


def test_oracle_matches_the_closed_form_and_library_matches_oracle():
    rng = np.random.default_rng(21)
    for _ in range(3000):
        cands, M, L = random_case(rng)
        ref = from_closed_form(cands, M, L)
        try:
            got_o = oracle.intra_select(cands, M, L)
        except Infeasible:
            got_o = None
        assert got_o == ref, (cands, M, L)
        try:
            got = B.dcp_intra_select(cands, M, L)
        except B.DcpError as e:
            assert e.code == B.DCP_ERR_INFEASIBLE
            got = None
        assert got == got_o, (cands, M, L)


def test_hand_worked_example():
    # L = 4 layers, capacity 100.  Profiled with all four layers recomputed:
    #   A: b=1, p=1, t_f=10, m=20, T=140, M=50 -> 2 layers fit (50 + 2*20 = 90), r = 2, time 120, throughput 1/120
    #   B: b=2, p=1, t_f=18, m=45, T=250, M=60 -> 0 layers fit (60 + 45 > 100), r = 4, time 250, throughput 2/250
    #   C: b=4, p=2, t_f=12, m=10, T=260, M=60 -> 4 layers fit (60 + 40 = 100), r = 0, time 212, throughput 4/424
    # 4/424 = 0.00943 > 1/120 = 0.00833 > 2/250 = 0.008 -> C
    cands = [(1, 1, 10, 20, 140, 50), (2, 1, 18, 45, 250, 60), (4, 2, 12, 10, 260, 60)]
    assert oracle.intra_select(cands, 100, 4) == (2, 0, 212)
    assert B.dcp_intra_select(cands, 100, 4) == (2, 0, 212)
    # one byte less: C keeps only 3 layers (time 224, 4/448 = 0.00893), still ahead of A
    assert B.dcp_intra_select(cands, 99, 4) == (2, 1, 224)
    # capacity 59: only A fits, with no spare memory -> full recompute
    assert B.dcp_intra_select(cands, 59, 4) == (0, 4, 140)
    assert oracle.intra_select(cands, 59, 4) == (0, 4, 140)


def test_equal_b_and_p_reduces_to_the_smallest_time():
    rng = np.random.default_rng(22)
    for _ in range(300):
        cands, M, L = random_case(rng)
        cands = [(3, 2) + c[2:] for c in cands]
        M = max(M, max(c[5] for c in cands))
        idx, r, t = B.dcp_intra_select(cands, M, L)
        assert oracle.intra_select(cands, M, L) == (idx, r, t)
        times = [c[4] - min(L, (M - c[5]) // c[3] if c[3] else L) * c[2] for c in cands]
        assert t == min(times) and idx == times.index(min(times))


def test_more_memory_never_hurts_and_enough_memory_removes_recompute():
    rng = np.random.default_rng(23)
    for _ in range(300):
        cands, M, L = random_case(rng)
        M = max(M, min(c[5] for c in cands))
        i0, r0, t0 = B.dcp_intra_select(cands, M, L)
        i1, r1, t1 = B.dcp_intra_select(cands, M + 500, L)
        assert Fraction(cands[i1][0], cands[i1][1] * t1) >= Fraction(cands[i0][0], cands[i0][1] * t0)
        big = max(c[5] + L * c[3] for c in cands)
        assert B.dcp_intra_select(cands, big, L)[1] == 0


def test_ties_and_errors():
    # same throughput 1/100 three ways: smaller p wins, then larger b
    cands = [(2, 2, 0, 0, 100, 0), (1, 1, 0, 0, 100, 0), (2, 1, 0, 0, 200, 0), (1, 1, 0, 0, 100, 0)]
    assert B.dcp_intra_select(cands, 10, 3)[0] == 2 and oracle.intra_select(cands, 10, 3)[0] == 2
    with pytest.raises(B.DcpError) as e:
        B.dcp_intra_select([(1, 1, 5, 5, 100, 50)], 49, 2)
    assert e.value.code == B.DCP_ERR_INFEASIBLE
    for bad in [(0, 1, 1, 1, 10, 1), (1, 0, 1, 1, 10, 1), (1, 1, -1, 1, 10, 1), (1, 1, 1, 1, 0, 1), (1, 1, 6, 0, 10, 1)]:
        with pytest.raises(B.DcpError) as e:
            B.dcp_intra_select([bad], 100, 2)
        assert e.value.code == B.DCP_ERR_INVALID_ARG
    with pytest.raises(B.DcpError):
        B.dcp_intra_select([], 100, 2)
