"""Pins for the fp64 attention oracle: closed forms, invariants, symmetries, finite differences and
an independent dense fp64 evaluation with CPU autograd.  None of these touches the CUDA path."""
import numpy as np
import pytest
import torch

import oracle
from paper_2608_07524_b200 import inputs


def bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round float values to bf16 and return the bit patterns."""
    t = torch.from_numpy(np.asarray(x, dtype=np.float32)).to(torch.bfloat16)
    return t.view(torch.int16).numpy().view(np.uint16).copy()


def bits_to_f64(b: np.ndarray) -> np.ndarray:
    return (b.astype(np.uint32) << 16).view(np.float32).astype(np.float64)


def rand_bits(rng, shape, scale=1.0):
    return bf16_bits(rng.standard_normal(shape) * scale)


def dense_reference(q, k, v, g, cu, causal, scale=None):
    """Per sequence and head: softmax(Q K^T s + mask) V in fp64 with torch CPU ops, gradients by
    autograd.  A library evaluation of the special case 'one dense sequence'."""
    T, H, d = q.shape
    s = (1.0 / np.sqrt(d)) if scale is None else scale
    Q = torch.tensor(bits_to_f64(q), requires_grad=True)
    K = torch.tensor(bits_to_f64(k), requires_grad=True)
    V = torch.tensor(bits_to_f64(v), requires_grad=True)
    G = torch.tensor(bits_to_f64(g))
    O = torch.zeros_like(Q)
    lse = torch.zeros((H, T), dtype=torch.float64)
    outs = []
    for b in range(len(cu) - 1):
        a, e = cu[b], cu[b + 1]
        if e == a:
            continue
        S = torch.einsum("ihc,jhc->hij", Q[a:e], K[a:e]) * s
        if causal:
            L = e - a
            mask = torch.ones(L, L, dtype=torch.bool).tril()
            S = S.masked_fill(~mask, float("-inf"))
        P = torch.softmax(S, dim=-1)
        outs.append((a, e, torch.einsum("hij,jhc->ihc", P, V[a:e]), torch.logsumexp(S, dim=-1)))
    loss = sum((o * G[a:e]).sum() for a, e, o, _ in outs)
    loss.backward()
    with torch.no_grad():
        for a, e, o, l in outs:
            O[a:e] = o
            lse[:, a:e] = l
    return (O.detach().numpy(), lse.numpy(), Q.grad.numpy(), K.grad.numpy(), V.grad.numpy())


@pytest.mark.parametrize("causal", [False, True])
def test_matches_dense_autograd_on_config1(causal):
    w = inputs.config(1, causal)
    q, k, v, g = inputs.make_qkvg(w.total_tokens, w.n_heads, w.head_dim, w.value_seed)
    qb, kb, vb, gb = (oracle._bits(x) for x in (q, k, v, g))
    O, lse = oracle.attn_fwd(qb, kb, vb, w.cu_seqlens, causal)
    dq, dk, dv = oracle.attn_bwd(qb, kb, vb, gb, w.cu_seqlens, causal)
    rO, rlse, rdq, rdk, rdv = dense_reference(qb, kb, vb, gb, w.cu_seqlens, causal)
    for name, a, b in (("O", O, rO), ("lse", lse, rlse), ("dq", dq, rdq), ("dk", dk, rdk), ("dv", dv, rdv)):
        assert np.max(np.abs(a - b)) < 1e-11, name


def test_custom_scale_and_zero_length_sequences():
    rng = np.random.default_rng(1)
    cu = [0, 0, 5, 5, 12, 12]
    q, k, v, g = (rand_bits(rng, (12, 3, 8)) for _ in range(4))
    for causal in (False, True):
        O, lse = oracle.attn_fwd(q, k, v, cu, causal, scale=0.3)
        dq, dk, dv = oracle.attn_bwd(q, k, v, g, cu, causal, scale=0.3)
        rO, rlse, rdq, rdk, rdv = dense_reference(q, k, v, g, cu, causal, scale=0.3)
        assert np.max(np.abs(O - rO)) < 1e-12 and np.max(np.abs(lse - rlse)) < 1e-12
        assert max(np.max(np.abs(dq - rdq)), np.max(np.abs(dk - rdk)), np.max(np.abs(dv - rdv))) < 1e-11


def test_length_one_closed_form():
    # L = 1: P = [1]; O = V, lse = s * q.k, dV = dO, dQ = dK = 0.
    rng = np.random.default_rng(2)
    q, k, v, g = (rand_bits(rng, (3, 2, 16)) for _ in range(4))
    cu = [0, 1, 2, 3]
    for causal in (False, True):
        O, lse = oracle.attn_fwd(q, k, v, cu, causal)
        dq, dk, dv = oracle.attn_bwd(q, k, v, g, cu, causal)
        assert np.array_equal(O, bits_to_f64(v))
        expect = np.einsum("thc,thc->ht", bits_to_f64(q), bits_to_f64(k)) / 4.0
        assert np.max(np.abs(lse - expect)) < 1e-14
        assert np.array_equal(dv, bits_to_f64(g))
        assert np.max(np.abs(dq)) == 0.0 and np.max(np.abs(dk)) == 0.0


def test_zero_queries_give_uniform_weights():
    # Q = 0: every visible key has weight 1/n, O = mean of visible V, lse = ln n.
    rng = np.random.default_rng(3)
    L, H, d = 37, 2, 8
    q = np.zeros((L, H, d), np.uint16)
    k, v = rand_bits(rng, (L, H, d)), rand_bits(rng, (L, H, d))
    V = bits_to_f64(v)
    O, lse = oracle.attn_fwd(q, k, v, [0, L], False)
    assert np.max(np.abs(O - V.mean(axis=0, keepdims=True))) < 1e-14
    assert np.max(np.abs(lse - np.log(L))) < 1e-14
    O, lse = oracle.attn_fwd(q, k, v, [0, L], True)
    prefix_mean = np.cumsum(V, axis=0) / np.arange(1, L + 1)[:, None, None]
    assert np.max(np.abs(O - prefix_mean)) < 1e-14
    assert np.max(np.abs(lse - np.log(np.arange(1, L + 1))[None, :])) < 1e-14


def test_identical_keys_give_mean_of_values_and_zero_dq():
    # All keys equal: scores are constant along a row, so P is uniform, O = mean(V); and because
    # every dS row sums to zero, dQ_i = s * (sum_j dS_ij) k0 = 0.
    rng = np.random.default_rng(4)
    L, H, d = 29, 2, 8
    q, v, g = (rand_bits(rng, (L, H, d)) for _ in range(3))
    k = np.repeat(rand_bits(rng, (1, H, d)), L, axis=0)
    O, _ = oracle.attn_fwd(q, k, v, [0, L], False)
    assert np.max(np.abs(O - bits_to_f64(v).mean(axis=0, keepdims=True))) < 1e-13
    dq, _, _ = oracle.attn_bwd(q, k, v, g, [0, L], False)
    assert np.max(np.abs(dq)) < 1e-13


def test_rows_of_p_sum_to_one():
    # V = 1 everywhere => O = 1 exactly when the weights of each row sum to one; and then
    # sum_j dV_j = sum_i dO_i for any V.
    rng = np.random.default_rng(5)
    L, H, d = 50, 2, 8
    q, k, g = (rand_bits(rng, (L, H, d), 2.0) for _ in range(3))
    ones = bf16_bits(np.ones((L, H, d)))
    for causal in (False, True):
        O, _ = oracle.attn_fwd(q, k, ones, [0, L], causal)
        assert np.max(np.abs(O - 1.0)) < 1e-14
        v = rand_bits(rng, (L, H, d))
        _, _, dv = oracle.attn_bwd(q, k, v, g, [0, L], causal)
        assert np.max(np.abs(dv.sum(axis=0) - bits_to_f64(g).sum(axis=0))) < 1e-12


def test_whole_tensor_identities():
    # sum_i <Q_i, dQ_i> = sum_j <K_j, dK_j>  (both equal sum_ij dS_ij S_ij) per sequence and head.
    w = inputs.config(1, True)
    q, k, v, g = (oracle._bits(x) for x in inputs.make_qkvg(w.total_tokens, 2, 64, 99))
    dq, dk, _ = oracle.attn_bwd(q, k, v, g, w.cu_seqlens, True)
    Q, K = bits_to_f64(q), bits_to_f64(k)
    for b in range(4):
        a, e = w.cu_seqlens[b], w.cu_seqlens[b + 1]
        lhs = np.einsum("thc,thc->h", Q[a:e], dq[a:e])
        rhs = np.einsum("thc,thc->h", K[a:e], dk[a:e])
        assert np.max(np.abs(lhs - rhs)) < 1e-10


def test_symmetries():
    rng = np.random.default_rng(6)
    L, H, d = 33, 2, 16
    q, k, v, g = (rand_bits(rng, (L, H, d)) for _ in range(4))
    O, lse = oracle.attn_fwd(q, k, v, [0, L], False)
    # scaling Q by 2 and K by 1/2 is exact in bf16 and changes nothing
    q2 = bf16_bits(bits_to_f64(q) * 2.0)
    kh = bf16_bits(bits_to_f64(k) * 0.5)
    O2, lse2 = oracle.attn_fwd(q2, kh, v, [0, L], False)
    assert np.max(np.abs(O - O2)) < 1e-14 and np.max(np.abs(lse - lse2)) < 1e-13
    # permuting keys and values together leaves a bidirectional O unchanged
    perm = rng.permutation(L)
    O3, lse3 = oracle.attn_fwd(q, k[perm], v[perm], [0, L], False)
    assert np.max(np.abs(O - O3)) < 1e-13 and np.max(np.abs(lse - lse3)) < 1e-13
    # adding one vector to every key shifts each row's scores by a constant: O unchanged
    kint = bf16_bits(np.round(bits_to_f64(k) * 4) / 4)          # few mantissa bits
    kshift = bf16_bits(bits_to_f64(kint) + 0.5)                 # still exact in bf16
    assert np.array_equal(bits_to_f64(kshift), bits_to_f64(kint) + 0.5)
    Oa, _ = oracle.attn_fwd(q, kint, v, [0, L], False)
    Ob, _ = oracle.attn_fwd(q, kshift, v, [0, L], False)
    assert np.max(np.abs(Oa - Ob)) < 1e-13


def test_packing_independence():
    # A sequence's results do not depend on its neighbours in the packed batch.
    rng = np.random.default_rng(7)
    H, d = 2, 16
    lens = [9, 20, 13]
    cu = np.concatenate([[0], np.cumsum(lens)])
    q, k, v, g = (rand_bits(rng, (cu[-1], H, d)) for _ in range(4))
    for causal in (False, True):
        O, lse = oracle.attn_fwd(q, k, v, cu, causal)
        dq, dk, dv = oracle.attn_bwd(q, k, v, g, cu, causal)
        a, e = cu[1], cu[2]
        O1, lse1 = oracle.attn_fwd(q[a:e], k[a:e], v[a:e], [0, lens[1]], causal)
        dq1, dk1, dv1 = oracle.attn_bwd(q[a:e], k[a:e], v[a:e], g[a:e], [0, lens[1]], causal)
        assert np.array_equal(O[a:e], O1) and np.array_equal(lse[:, a:e], lse1)
        assert np.array_equal(dq[a:e], dq1) and np.array_equal(dk[a:e], dk1) and np.array_equal(dv[a:e], dv1)
        # changing the neighbours' data changes nothing either
        q2, k2, v2 = q.copy(), k.copy(), v.copy()
        for x in (q2, k2, v2):
            x[:a] = rand_bits(rng, (a, H, d))
            x[e:] = rand_bits(rng, (cu[-1] - e, H, d))
        O2, _ = oracle.attn_fwd(q2, k2, v2, cu, causal)
        assert np.array_equal(O[a:e], O2[a:e])


@pytest.mark.parametrize("causal", [False, True])
def test_finite_differences(causal):
    """Central differences with Richardson extrapolation on a grid of bf16-exact inputs.
    Inputs are multiples of 1/8 in [-1.875, 1.875]; steps 2^-6 and 2^-7 keep every perturbed
    value exactly representable in bf16, so the loss is evaluated at the intended points."""
    rng = np.random.default_rng(8)
    L, H, d = 6, 2, 4
    cu = [0, L]

    def grid(shape):
        return rng.integers(-15, 16, size=shape).astype(np.float64) / 8.0

    X = {n: grid((L, H, d)) for n in "qkvg"}

    def loss(x):
        b = {n: bf16_bits(x[n]) for n in "qkvg"}
        for n in "qkvg":
            assert np.array_equal(bits_to_f64(b[n]), x[n])      # nothing was rounded
        O, _ = oracle.attn_fwd(b["q"], b["k"], b["v"], cu, causal)
        return float(np.sum(O * x["g"]))

    b = {n: bf16_bits(X[n]) for n in "qkvg"}
    grads = dict(zip("qkv", oracle.attn_bwd(b["q"], b["k"], b["v"], b["g"], cu, causal)))
    for name in "qkv":
        for idx in np.ndindex(L, H, d):
            def cd(h):
                xp = {n: a.copy() for n, a in X.items()}
                xm = {n: a.copy() for n, a in X.items()}
                xp[name][idx] += h
                xm[name][idx] -= h
                return (loss(xp) - loss(xm)) / (2 * h)
            h = 2.0 ** -6
            fd = (4.0 * cd(h / 2) - cd(h)) / 3.0
            assert abs(fd - grads[name][idx]) < 2e-6, (name, idx, fd, grads[name][idx])


@pytest.mark.parametrize("causal", [False, True])
def test_sampled_rows_and_columns_equal_the_full_result(causal):
    rng = np.random.default_rng(9)
    lens = [70, 130]
    cu = [0, 70, 200]
    H, d = 3, 16
    q, k, v, g = (rand_bits(rng, (200, H, d)) for _ in range(4))
    O, lse = oracle.attn_fwd(q, k, v, cu, causal)
    dq, dk, dv = oracle.attn_bwd(q, k, v, g, cu, causal)
    rows = np.array([0, 1, 63, 64, 127, 128, 129], np.int32)
    Or, lr, dqr = oracle.attn_rows(q, k, v, g, cu, causal, 1, 2, rows)
    assert np.max(np.abs(Or - O[70 + rows, 2])) < 1e-14
    assert np.max(np.abs(lr - lse[2, 70 + rows])) < 1e-14
    assert np.max(np.abs(dqr - dq[70 + rows, 2])) < 1e-13
    cols = np.array([5, 64, 100, 129], np.int32)
    dkc, dvc = oracle.attn_cols(q, k, v, g, cu, causal, 1, 2, cols)
    assert np.max(np.abs(dkc - dk[70 + cols, 2])) < 1e-13
    assert np.max(np.abs(dvc - dv[70 + cols, 2])) < 1e-13
    # and against the dense autograd evaluation directly
    rO, rlse, rdq, rdk, rdv = dense_reference(q, k, v, g, cu, causal)
    assert np.max(np.abs(Or - rO[70 + rows, 2])) < 1e-12
    assert np.max(np.abs(dkc - rdk[70 + cols, 2])) < 1e-12
    assert np.max(np.abs(dvc - rdv[70 + cols, 2])) < 1e-12
    assert np.max(np.abs(dqr - rdq[70 + rows, 2])) < 1e-12
