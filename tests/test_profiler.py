"""Profiled planning (Section 3.5 feeding Eq. 5): the planner with measured per-sequence forward
times against the brute-force oracle, and the host logic of the dual-layer profiler."""
import numpy as np
import pytest

import oracle
from paper_2608_07524_b200 import binding as B
from oracle import profile_oracle
from paper_2608_07524_b200.profiler import ProfileTable, dual_layer_profile, intra_candidates, select_group_setting
from paper_2608_07524_b200.stream import plan_batch


def both(lengths, fwd_time, budget, **kw):
    try:
        ref = oracle.plan_bruteforce(lengths, budget, fwd_time=fwd_time, **kw)
    except oracle.Infeasible:
        ref = None
    try:
        got = B.dcp_plan_profiled(lengths, fwd_time, budget, **kw)
    except B.DcpError as e:
        assert e.code == B.DCP_ERR_INFEASIBLE
        got = None
    return got, ref


def test_profiled_planner_matches_bruteforce_on_random_cases():
    rng = np.random.default_rng(5)
    for _ in range(3000):
        n = int(rng.integers(1, 11))
        lengths = [int(x) for x in rng.integers(1, 500, size=n)]
        # times unrelated to length on purpose: the planner may not assume any shape of t_f(L)
        fwd_time = [int(x) for x in rng.integers(0, 10 ** int(rng.integers(1, 12)), size=n)]
        lam = int(rng.choice([1, 2, 4, 28]))
        TC = int(rng.choice([0, 1, 50, 10 ** 5, 1 << 24, 1 << 40]))
        unit = 2 * 8 * 2
        budget = int(rng.integers(max(lam * unit * max(lengths) - 40, 0), 5 * lam * unit * sum(lengths) + 2))
        got, ref = both(lengths, fwd_time, budget, n_heads=2, head_dim=8, n_layers=lam, fixed_cost=TC)
        assert got == ref, (lengths, fwd_time, budget, lam, TC)


def test_profiled_with_model_times_equals_model_planner():
    rng = np.random.default_rng(6)
    for _ in range(500):
        n = int(rng.integers(1, 20))
        lengths = [int(x) for x in rng.integers(1, 3000, size=n)]
        lam = int(rng.choice([1, 3, 28]))
        budget = int(rng.integers(lam * 32 * max(lengths), 5 * lam * 32 * sum(lengths) + 2))
        kw = dict(n_heads=2, head_dim=8, n_layers=lam, fixed_cost=12345)
        assert B.dcp_plan_profiled(lengths, [2 * L * L for L in lengths], budget, **kw) == B.dcp_plan(lengths, budget, **kw)


def test_hand_worked_case():
    # two sequences of 10 tokens, H = d = e = 1, Lambda = 1: mem(r) of a block = (1 - r) 4 tok + tok.
    # budget 60: both together need 100 at r = 0 and 20 at r = 1, so r = 1; alone each needs 50, r = 0.
    # together costs T_C + 1 * (7 + 5), split costs 2 T_C: split wins iff T_C < 12, a tie goes to fewer blocks.
    kw = dict(n_heads=1, head_dim=1, elt_bytes=1, n_layers=1)
    assert B.dcp_plan_profiled([10, 10], [7, 5], 60, fixed_cost=11, **kw) == ([0, 1], [0, 0], 22)
    assert B.dcp_plan_profiled([10, 10], [7, 5], 60, fixed_cost=13, **kw) == ([0, 0], [1], 25)
    assert B.dcp_plan_profiled([10, 10], [7, 5], 60, fixed_cost=12, **kw) == ([0, 0], [1], 24)   # tie: fewer blocks
    assert oracle.plan_bruteforce([10, 10], 60, fixed_cost=12, fwd_time=[7, 5], **kw) == ([0, 0], [1], 24)


def test_profiled_argument_errors():
    with pytest.raises(B.DcpError) as e:
        B.dcp_plan_profiled([5, 6], [1, -1], 10 ** 9)
    assert e.value.code == B.DCP_ERR_INVALID_ARG
    with pytest.raises(ValueError):
        B.dcp_plan_profiled([5, 6], [1], 10 ** 9)
    with pytest.raises(B.DcpError) as e:
        B.dcp_plan_profiled([5, 6], [2 ** 62, 2 ** 62], 16 * 128 * 2 * 11 + 1, n_layers=2, fixed_cost=2 ** 62)
    assert e.value.code in (B.DCP_ERR_OVERFLOW, B.DCP_ERR_INFEASIBLE)


def test_interpolation_oracle_hand_values():
    # pins of the plain-Python oracle: values worked by hand from the rule (linear below the first bucket,
    # linear between buckets, quadratic above the last, floor division)
    xs, f, b = [100, 200, 400], [1000, 3000, 11000], [2000, 7000, 30000]
    o = profile_oracle.interp
    assert [o(xs, f, L) for L in (100, 200, 400)] == [1000, 3000, 11000]
    assert o(xs, f, 50) == 500 and o(xs, f, 1) == 10                   # 1000 * L / 100
    assert o(xs, f, 150) == 2000 and o(xs, f, 201) == 3040             # 3000 + 8000 * 1 / 200
    assert o(xs, f, 800) == 44000 and o(xs, f, 401) == 11000 * 401 * 401 // 160000
    assert o(xs, b, 300) == 18500
    vals = [o(xs, f, L) for L in range(1, 1000)]
    assert all(y >= x for x, y in zip(vals, vals[1:]))
    assert o([10, 20], [9, 2], 13) == 6                                # falling table: 9 + floor(-7 * 3 / 10) = 9 - 3
    # Eq. 4-5: Lambda (t_f + t_b) + r t_f + T_C; at r = Lambda it is Section 3.5's Lambda (2 t_f + t_b) + T_C
    assert profile_oracle.model_time([1000, 3000], [2000, 7000], 3, 2, 7) == 3 * (4000 + 9000) + 2 * 4000 + 7
    assert profile_oracle.model_time([5], [11], 4, 4, 9) == 4 * (2 * 5 + 11) + 9
    assert profile_oracle.candidate(2, 1, 5, 11, 40, 10, 4, 3, 9) == (2, 1, 5, 40, 4 * (2 * 5 + 11) + 9, 4 * 10 + 3)


def test_library_interpolation_and_model_time_match_the_oracle():
    t = ProfileTable([100, 200, 400], [1000, 3000, 11000], [2000, 7000, 30000], [1, 2, 4])
    assert t.fwd_time(150) == 2000 and t.bwd_time(300) == 18500 and t.fwd_time(800) == 44000
    rng = np.random.default_rng(31)
    for _ in range(300):
        nb = int(rng.integers(1, 8))
        xs = sorted(set(int(x) for x in rng.integers(1, 5000, size=nb)))
        ys = [int(x) for x in rng.integers(0, 10 ** int(rng.integers(1, 12)), size=len(xs))]
        ls = [int(x) for x in rng.integers(1, 9000, size=20)] + xs
        assert B.dcp_profile_interp(xs, ys, ls) == [profile_oracle.interp(xs, ys, L) for L in ls]
        f = [int(x) for x in rng.integers(0, 10 ** 9, size=6)]
        b = [int(x) for x in rng.integers(0, 10 ** 9, size=6)]
        lam = int(rng.integers(1, 40))
        r = int(rng.integers(0, lam + 1))
        assert B.dcp_model_time(f, b, lam, r, 12345) == profile_oracle.model_time(f, b, lam, r, 12345)
        args = (int(rng.integers(1, 9)), 1, f[0], b[0], f[1], f[2], lam, f[3], f[4])
        assert B.dcp_intra_candidate_from_profile(*args) == profile_oracle.candidate(*args)
    assert t.model_time([100, 200], 3, 2, 7) == 3 * (4000 + 9000) + 2 * 4000 + 7
    # memory model of a micro-batch (config 5: 4 * L * H * d * 2 bytes of activations per sequence) and the
    # grouping of a length group into micro-batches of b sequences
    assert B.dcp_activation_bytes(1000, 16, 128) == (4 * 1000 * 16 * 128 * 2, 1000 * 16 * 128 * 2)
    assert B.dcp_activation_bytes(0, 1, 8, 4) == (0, 0)
    assert B.dcp_length_group_plan(7, 3) == ([0, 0, 0, 1, 1, 1, 2], 3) and B.dcp_length_group_plan(4, 8) == ([0] * 4, 1)
    with pytest.raises(B.DcpError):
        B.dcp_length_group_plan(0, 3)
    with pytest.raises(ValueError):
        ProfileTable([100, 100], [1, 2], [1, 2], [1, 2])
    with pytest.raises(B.DcpError) as e:
        t.fwd_time(0)
    assert e.value.code == B.DCP_ERR_INVALID_ARG
    with pytest.raises(B.DcpError):
        B.dcp_profile_interp([5, 5], [1, 2], [3])
    with pytest.raises(B.DcpError) as e:
        B.dcp_profile_interp([5], [2 ** 62], [500])
    assert e.value.code == B.DCP_ERR_OVERFLOW


def test_algorithm_1_table_from_a_fake_profile():
    # forward 1 ms per sequence of the batch, backward 3 ms, whatever b: per-sequence time is flat, so the
    # throughput b / T is the same for every b and only memory decides how many layers are recomputed
    runs = []

    def fake_layer(lengths):
        runs.append(len(lengths))
        return 1.0 * len(lengths), 3.0 * len(lengths)

    H, d, L, lam = 4, 32, 1000, 6
    cands = intra_candidates(L, [1, 2, 4], H, d, False, lam, run_layer=fake_layer, fixed_cost_ns=500)
    assert runs == [1, 1, 2, 2, 4, 4]                                    # warm-up + recorded run per batch size
    unit = L * H * d * 2
    assert cands == [profile_oracle.candidate(b, 1, b * 10 ** 6, 3 * b * 10 ** 6, 4 * b * unit, b * unit, lam, 0, 500)
                     for b in (1, 2, 4)]
    # capacity for b = 4 with no layer kept, b = 2 with one kept, b = 1 with all six kept
    cap = lam * 4 * unit
    b, r, t = select_group_setting(cands, cap, lam)
    assert (b, r, t) == (lambda i, rr, tt: (cands[i][0], rr, tt))(*oracle.intra_select(cands, cap, lam))
    # b = 1 keeps floor((24 - 6) / 4) = 4 layers: T = 6 * 5 ms + 500 - 4 * 1 ms = 26 ms + 500 ns per sequence;
    # b = 2 keeps (24 - 12) / 8 = 1: (60 ms + 500 - 2 ms) / 2 = 29 ms; b = 4 keeps none: 30 ms per sequence
    assert (b, r, t) == (1, 2, 26 * 10 ** 6 + 500)


def test_dual_layer_profile_keeps_the_second_run():
    calls = []

    def fake_layer(lengths):
        calls.append(list(lengths))
        first = sum(1 for c in calls if c == list(lengths)) == 1
        L, n = lengths[0], len(lengths)
        return (999.0, 999.0) if first else (n * L * L * 1e-6, n * L * L * 3e-6)   # ms

    t = dual_layer_profile([256, 64, 1024], n_heads=4, head_dim=32, causal=False, fill_tokens=1024, run_layer=fake_layer)
    assert t.lengths == [64, 256, 1024]
    assert [len(c) for c in calls] == [16, 16, 4, 4, 1, 1]          # batches hold about fill_tokens tokens
    assert t.t_f_ns == [64 * 64, 256 * 256, 1024 * 1024]            # per sequence, ns; warm-up discarded
    assert t.t_b_ns == [3 * x for x in t.t_f_ns]
    assert t.m_bytes == [4 * L * 4 * 32 * 2 for L in t.lengths]


def test_plan_batch_with_profile_uses_measured_times():
    # a table in which recomputing is nearly free makes one micro-batch with recompute the best plan;
    # one in which it is expensive makes the planner split instead
    lengths = [4000, 3000, 2000, 1000]
    unit = 16 * 128 * 2
    budget = 3 * unit * sum(lengths)              # all four together only fit when recomputed
    cheap = ProfileTable([1000, 4000], [1, 4], [1, 4], [1, 1])
    dear = ProfileTable([1000, 4000], [10 ** 6, 16 * 10 ** 6], [1, 4], [1, 1])
    one = plan_batch(lengths, budget, 16, 128, n_layers=1, fixed_cost=1000, profile=cheap).micro_batches
    assert [list(m.lengths) for m in one] == [lengths] and one[0].recompute == 1 and one[0].seg is None
    many = plan_batch(lengths, budget, 16, 128, n_layers=1, fixed_cost=1000, profile=dear).micro_batches
    assert len(many) == 2 and all(m.recompute == 0 for m in many)
    assert sorted(sum((list(m.lengths) for m in many), [])) == sorted(lengths)


@pytest.mark.gpu
def test_profile_on_device_and_plan():
    t = dual_layer_profile([512, 2048, 8192], n_heads=16, head_dim=128, causal=False, fill_tokens=1 << 15)
    assert all(x > 0 for x in t.t_f_ns + t.t_b_ns)
    assert t.t_f_ns[0] < t.t_f_ns[1] < t.t_f_ns[2] and t.t_b_ns[0] < t.t_b_ns[1] < t.t_b_ns[2]
    # the kernels are quadratic in length once tensor-bound: 4x the length costs 8-20x the time
    assert 8 < t.t_f_ns[2] / t.t_f_ns[1] < 20
    assert all(b > f for f, b in zip(t.t_f_ns, t.t_b_ns))
    lengths = [9600, 9600, 3600, 2048, 1024, 256]
    plan = plan_batch(lengths, 5 * 16 * 128 * 2 * 14000, 16, 128, n_layers=1, fixed_cost=20000, profile=t)
    assert sorted(sum((list(m.lengths) for m in plan.micro_batches), [])) == sorted(lengths)
    ref = oracle.plan_bruteforce(lengths, 5 * 16 * 128 * 2 * 14000, fixed_cost=20000,
                                 fwd_time=[profile_oracle.interp(t.lengths, t.t_f_ns, L) for L in lengths])
    assert (plan.mb_id, plan.recompute, plan.cost) == ref
