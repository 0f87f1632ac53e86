"""Parity of the CUDA attention path (through the C ABI) against the fp64 CPU oracle.

Tolerances (bf16 outputs upcast to fp64, both must hold per tensor):
    max-abs <= 5e-2  and  ||x - ref||_F / ||ref||_F <= 1e-2;   lse (fp32): max-abs <= 2e-3.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2608_07524_b200 import binding as B
from paper_2608_07524_b200 import inputs

pytestmark = pytest.mark.gpu

MAX_ABS, REL_FRO, LSE_ABS = 5e-2, 1e-2, 2e-3


def to64(x):
    return x.detach().double().cpu().numpy()


def assert_close(name, got, ref):
    got = to64(got) if torch.is_tensor(got) else got
    assert got.shape == ref.shape, name
    assert np.all(np.isfinite(got)), f"{name}: non-finite values"
    max_abs = float(np.max(np.abs(got - ref))) if ref.size else 0.0
    rel = float(np.linalg.norm(got - ref) / max(np.linalg.norm(ref), 1e-30)) if ref.size else 0.0
    assert max_abs <= MAX_ABS and rel <= REL_FRO, f"{name}: max-abs {max_abs:.3e}, rel-Frobenius {rel:.3e}"


GUARD_ROWS, GUARD_BYTES, GUARD_FILL = 128, 1 << 16, 0x5A


class Guarded:
    """Device buffers with a poisoned margin after their end: whatever a kernel stores past the last row
    of an output, past the end of lse or past the end of the workspace lands in the margin and is seen."""

    def __init__(self, T, H, d, n_seqs, dev):
        self.T, self.H, self.d = T, H, d
        row = H * d
        self.bf16 = [torch.full(((T + GUARD_ROWS) * row,), GUARD_FILL * 257, dtype=torch.int16, device=dev) for _ in range(4)]
        self.o, self.dq, self.dk, self.dv = (b[: T * row].view(torch.bfloat16).view(T, H, d) for b in self.bf16)
        self.lse_raw = torch.full((H * T + GUARD_BYTES // 4,), GUARD_FILL * 0x01010101, dtype=torch.int32, device=dev)
        self.lse = self.lse_raw[: H * T].view(torch.float32).view(H, T)
        _, bwd = B.dcp_varlen_attn_workspace(T, n_seqs, H, d)
        self.ws_bytes = bwd
        self.ws_raw = torch.full((bwd + GUARD_BYTES,), GUARD_FILL, dtype=torch.uint8, device=dev)
        self.ws = self.ws_raw[:bwd]

    def assert_margins_untouched(self, what):
        row = self.H * self.d
        for name, b in zip(("o", "dq", "dk", "dv"), self.bf16):
            assert bool((b[self.T * row:] == GUARD_FILL * 257).all()), f"{what}: store past the end of {name}"
        assert bool((self.lse_raw[self.H * self.T:] == GUARD_FILL * 0x01010101).all()), f"{what}: store past the end of lse"
        assert bool((self.ws_raw[self.ws_bytes:] == GUARD_FILL).all()), f"{what}: store past the end of the workspace"


def run_gpu(q, k, v, g, cu, causal, scale=0.0, o_override=None, lse_override=None):
    dev = "cuda"
    cud = torch.tensor(np.asarray(cu), dtype=torch.int32, device=dev)
    lens = np.diff(np.asarray(cu))
    max_len = int(lens.max()) if lens.size else 0
    qd, kd, vd, gd = (x.to(dev) for x in (q, k, v, g))
    T, H, d = q.shape
    buf = Guarded(T, H, d, len(lens), dev)
    o, lse = B.dcp_varlen_attn_fwd(qd, kd, vd, cud, max_len, causal, scale, out=buf.o, lse=buf.lse, workspace=buf.ws)
    B.dcp_query_status(buf.ws)
    buf.assert_margins_untouched("forward")
    o_in = o if o_override is None else o_override.to(dev)
    lse_in = lse if lse_override is None else lse_override.to(dev)
    dq, dk, dv = B.dcp_varlen_attn_bwd(qd, kd, vd, o_in, gd, lse_in, cud, max_len, causal, scale, dq=buf.dq, dk=buf.dk,
                                       dv=buf.dv, workspace=buf.ws)
    B.dcp_query_status(buf.ws)
    buf.assert_margins_untouched("backward")
    return o, lse, dq, dk, dv


def check_full(lengths, H, d, causal, seed, scale=0.0):
    cu = np.concatenate([[0], np.cumsum(lengths)]).astype(np.int32)
    q, k, v, g = inputs.make_qkvg(int(cu[-1]), H, d, seed)
    o, lse, dq, dk, dv = run_gpu(q, k, v, g, cu, causal, scale)
    O, L = oracle.attn_fwd(q, k, v, cu, causal, scale)
    rdq, rdk, rdv = oracle.attn_bwd(q, k, v, g, cu, causal, scale)
    assert_close("o", o, O)
    assert float(np.max(np.abs(to64(lse) - L))) <= LSE_ABS if L.size else True
    assert_close("dq", dq, rdq)
    assert_close("dk", dk, rdk)
    assert_close("dv", dv, rdv)


@pytest.mark.parametrize("causal", [False, True])
def test_config1_tiny(causal):
    w = inputs.config(1, causal)
    check_full(w.lengths, w.n_heads, w.head_dim, causal, w.value_seed)


@pytest.mark.parametrize("causal", [False, True])
@pytest.mark.parametrize("d", [64, 128])
def test_ragged_multi_tile(causal, d):
    # several tiles, ragged tails on both the query and the key side, tile-edge lengths
    check_full([300, 1000, 129, 128, 1, 513, 127, 256, 257], 3, d, causal, seed=1)


@pytest.mark.parametrize("causal", [False, True])
def test_zero_length_sequences_and_single_tokens(causal):
    check_full([0, 5, 0, 0, 1, 130, 0], 2, 64, causal, seed=2)


def test_all_sequences_empty():
    q = torch.empty((0, 2, 64), dtype=torch.bfloat16)
    o, lse, dq, dk, dv = run_gpu(q, q, q, q, [0, 0, 0], False)
    assert o.numel() == 0 and dq.numel() == 0


@pytest.mark.parametrize("causal", [False, True])
def test_custom_softmax_scale(causal):
    check_full([200, 77], 2, 128, causal, seed=3, scale=0.05)


@pytest.mark.parametrize("causal", [False, True])
def test_many_short_sequences(causal):
    rng = np.random.default_rng(5)
    check_full([int(x) for x in rng.integers(1, 200, size=300)], 2, 64, causal, seed=5)


@pytest.fixture(params=["short-sequence kernels", "tile kernels"])
def both_paths(request):
    """Batches whose longest sequence has at most 32 tokens take the per-sequence kernels by default; the tile
    kernels (merged runs of short sequences) must keep handling them too."""
    B.dcp_set_short_sequence_path(request.param == "short-sequence kernels")
    yield request.param
    B.dcp_set_short_sequence_path(True)


@pytest.mark.parametrize("causal", [False, True])
@pytest.mark.parametrize("d", [64, 128])
def test_merged_tiny_sequences(causal, d, both_paths):
    # a 2-D model's temporal axis: thousands of sequences of 1-13 tokens, several of which share one tile
    rng = np.random.default_rng(11)
    check_full([int(x) for x in rng.choice([1, 4, 8, 13], size=700)], 2, d, causal, seed=11)


@pytest.mark.parametrize("causal", [False, True])
@pytest.mark.parametrize("H,d", [(4, 128), (16, 128), (2, 64), (3, 72), (1, 8), (6, 40), (12, 104), (4, 120), (5, 16)])
@pytest.mark.parametrize("max_len", [2, 13, 16, 17, 32])
def test_short_sequence_kernels(causal, H, d, max_len):
    """One CTA per (sequence, group of heads): every head-group width (4, 2, 1 heads), head dimensions with and
    without a last half k-step, one and two 16-row blocks, empty sequences, the longest allowed sequence."""
    rng = np.random.default_rng(1000 * max_len + H)
    lengths = [int(x) for x in rng.integers(0, max_len + 1, size=150)] + [max_len, 0, max_len, 1]
    check_full(lengths, H, d, causal, seed=50 + max_len, scale=0.0 if d != 40 else 0.2)


@pytest.mark.parametrize("causal", [False, True])
def test_short_sequence_kernels_on_single_tokens(causal):
    # closed form for L = 1: O = V, lse = the one score, dV = dO, dQ = dK = 0
    dev = "cuda"
    T, H, d = 500, 4, 128
    q, k, v, g = (x.to(dev) for x in inputs.make_qkvg(T, H, d, 3))
    cu = torch.arange(T + 1, dtype=torch.int32, device=dev)
    o, lse = B.dcp_varlen_attn_fwd(q, k, v, cu, 1, causal)
    dq, dk, dv = B.dcp_varlen_attn_bwd(q, k, v, o, g, lse, cu, 1, causal)
    assert torch.equal(o, v) and torch.equal(dv, g)
    score = (q.double() * k.double()).sum(-1) / d ** 0.5
    assert float((lse.double() - score.t()).abs().max()) <= 1e-4
    assert float(dq.float().abs().max()) <= 1e-4 and float(dk.float().abs().max()) <= 1e-4


@pytest.mark.parametrize("causal", [False, True])
def test_short_sequence_kernels_agree_with_the_tile_kernels(causal):
    dev = "cuda"
    rng = np.random.default_rng(77)
    lengths = [int(x) for x in rng.integers(1, 14, size=3000)]
    cu = np.concatenate([[0], np.cumsum(lengths)]).astype(np.int32)
    T, H, d = int(cu[-1]), 8, 128
    q, k, v, g = (x.to(dev) for x in inputs.make_qkvg(T, H, d, 78))
    cud = torch.tensor(cu, device=dev)
    out = []
    for short in (True, False):
        B.dcp_set_short_sequence_path(short)
        try:
            o, lse = B.dcp_varlen_attn_fwd(q, k, v, cud, 13, causal)
            out.append((o, lse) + tuple(B.dcp_varlen_attn_bwd(q, k, v, o, g, lse, cud, 13, causal)))
        finally:
            B.dcp_set_short_sequence_path(True)
    for name, a, b in zip(("o", "lse", "dq", "dk", "dv"), *out):
        # both are within tolerance of the oracle; against each other, a bf16 unit in the last place of the largest values
        assert float((a.float() - b.float()).abs().max()) <= (MAX_ABS if name != "lse" else 1e-4), name


def test_short_sequence_kernels_refuse_a_sequence_longer_than_declared():
    dev = "cuda"
    cu = torch.tensor([0, 5, 14, 20], dtype=torch.int32, device=dev)          # the middle sequence has 9 tokens
    q, k, v, g = (x.to(dev) for x in inputs.make_qkvg(20, 4, 64, 5))
    buf = Guarded(20, 4, 64, 3, dev)
    before = [b.clone() for b in buf.bf16]
    B.dcp_varlen_attn_fwd(q, k, v, cu, 8, False, out=buf.o, lse=buf.lse, workspace=buf.ws)
    with pytest.raises(B.DcpError) as e:
        B.dcp_query_status(buf.ws)
    assert e.value.code == B.DCP_ERR_INVALID_ARG
    B.dcp_varlen_attn_bwd(q, k, v, q, g, torch.zeros(4, 20, device=dev), cu, 8, False, dq=buf.dq, dk=buf.dk, dv=buf.dv,
                          workspace=buf.ws)
    with pytest.raises(B.DcpError):
        B.dcp_query_status(buf.ws)
    assert all(torch.equal(a, b) for a, b in zip(before, buf.bf16))           # nothing was computed
    B.dcp_varlen_attn_fwd(q, k, v, cu, 9, False, out=buf.o, lse=buf.lse, workspace=buf.ws)      # declared correctly: fine
    B.dcp_query_status(buf.ws)


@pytest.mark.parametrize("causal", [False, True])
def test_merged_mixed_with_long_and_empty(causal):
    # merged runs are broken by long, empty and medium sequences; lengths around the merge limit (64)
    # and the tile size; a run that fills a tile exactly
    lengths = [3, 5, 0, 7, 300, 1, 1, 1, 64, 64, 65, 63, 2, 128, 9, 0, 0, 4, 127, 13, 13, 13, 13, 13, 13, 13, 13, 13,
               11, 129, 6, 6, 6, 6, 100, 2, 2, 60, 60, 8, 32, 32, 32, 32, 1]
    check_full(lengths, 3, 128, causal, seed=12)


def test_merged_all_single_tokens():
    # every sequence has one token: O = V, dV = dO, dQ = dK = 0 whatever the packing
    n = 1000
    cu = np.arange(n + 1, dtype=np.int32)
    q, k, v, g = inputs.make_qkvg(n, 2, 64, 13)
    o, lse, dq, dk, dv = run_gpu(q, k, v, g, cu, False)
    assert torch.equal(o.cpu(), v) and torch.equal(dv.cpu(), g)
    # dS = P (dP - D) with dP = D up to fp32 rounding of two different summation orders
    assert float(dq.float().abs().max()) <= 1e-4 and float(dk.float().abs().max()) <= 1e-4
    ref_lse = (q.double() * k.double()).sum(-1).T.numpy() / 8.0
    assert float(np.max(np.abs(to64(lse) - ref_lse))) <= LSE_ABS


def test_merged_packing_independence():
    # neighbours inside the same merged tile must not leak into each other
    lengths = [10, 13, 7, 20, 13]
    cu = np.concatenate([[0], np.cumsum(lengths)]).astype(np.int32)
    q, k, v, g = inputs.make_qkvg(int(cu[-1]), 2, 128, 14)
    a = run_gpu(q, k, v, g, cu, False)
    gen = torch.Generator().manual_seed(4321)
    for _ in range(20):
        q2, k2, v2, g2 = (x.clone() for x in (q, k, v, g))
        for x in (q2, k2, v2, g2):
            x[:23] = (torch.randn(x[:23].shape, generator=gen) * 3).to(torch.bfloat16)
            x[30:] = (torch.randn(x[30:].shape, generator=gen) * 3).to(torch.bfloat16)
        b = run_gpu(q2, k2, v2, g2, cu, False)
        for i in (0, 2, 3, 4):      # a single tile pair: no atomics, dq is bit-exact too
            assert torch.equal(a[i][23:30], b[i][23:30])
        assert torch.equal(a[1][:, 23:30], b[1][:, 23:30])


def test_more_sequences_than_one_sorting_block():
    # above 1024 sequences the work list is ranked by a separate multi-CTA kernel
    rng = np.random.default_rng(6)
    check_full([int(x) for x in rng.integers(0, 60, size=1500)], 1, 64, True, seed=6)


@pytest.mark.parametrize("causal", [False, True])
def test_backward_in_isolation(causal):
    """Backward fed with the oracle's own O (rounded to bf16) and lse (fp32) instead of the GPU
    forward's, so a forward error cannot hide or cause a backward one."""
    lengths = [384, 100, 250]
    cu = np.concatenate([[0], np.cumsum(lengths)]).astype(np.int32)
    q, k, v, g = inputs.make_qkvg(int(cu[-1]), 2, 128, 7)
    O, L = oracle.attn_fwd(q, k, v, cu, causal)
    o_in = torch.from_numpy(O).to(torch.bfloat16)
    lse_in = torch.from_numpy(L).to(torch.float32)
    _, _, dq, dk, dv = run_gpu(q, k, v, g, cu, causal, o_override=o_in, lse_override=lse_in)
    rdq, rdk, rdv = oracle.attn_bwd(q, k, v, g, cu, causal)
    assert_close("dq", dq, rdq)
    assert_close("dk", dk, rdk)
    assert_close("dv", dv, rdv)


def test_packing_independence_on_gpu():
    """A sequence's outputs do not change when its neighbours' data change (tail tiles read the
    next sequence's rows through TMA, so the masks must hide them completely, and no decision a row
    takes may depend on the other rows of its warp).  Many neighbour draws: a dependence through the
    lazy rescale of the running maximum only shows for a few per cent of them."""
    lengths = [100, 200, 150]
    cu = np.concatenate([[0], np.cumsum(lengths)]).astype(np.int32)
    q, k, v, g = inputs.make_qkvg(int(cu[-1]), 2, 128, 9)
    a = run_gpu(q, k, v, g, cu, False)
    gen = torch.Generator().manual_seed(1234)
    for _ in range(60):
        q2, k2, v2, g2 = (x.clone() for x in (q, k, v, g))
        for x in (q2, k2, v2, g2):
            x[:100] = (torch.randn(x[:100].shape, generator=gen) * 3).to(torch.bfloat16)
            x[300:] = (torch.randn(x[300:].shape, generator=gen) * 3).to(torch.bfloat16)
        b = run_gpu(q2, k2, v2, g2, cu, False)
        for i in (0, 2, 3, 4):     # o, dq, dk, dv: this sequence has two key blocks, and a + b = b + a in fp32
            assert torch.equal(a[i][100:300], b[i][100:300])
        assert torch.equal(a[1][:, 100:300], b[1][:, 100:300])


def test_library_rejects_bad_arguments():
    dev = "cuda"
    q = torch.zeros((10, 2, 100), dtype=torch.bfloat16, device=dev)       # not a multiple of 8
    cu = torch.tensor([0, 10], dtype=torch.int32, device=dev)
    with pytest.raises(B.DcpError) as e:
        B.dcp_varlen_attn_fwd(q, q, q, cu, 10, False)
    assert e.value.code == B.DCP_ERR_UNSUPPORTED
    q = torch.zeros((10, 2, 64), dtype=torch.bfloat16, device=dev)
    small = torch.empty(16, dtype=torch.uint8, device=dev)
    with pytest.raises(B.DcpError) as e:
        B.dcp_varlen_attn_fwd(q, q, q, cu, 10, False, workspace=small)
    assert e.value.code == B.DCP_ERR_WORKSPACE
    with pytest.raises(B.DcpError) as e:
        B.dcp_varlen_attn_fwd(q, q, q, cu, 10, False, softmax_scale=-1.0)
    assert e.value.code == B.DCP_ERR_INVALID_ARG
    with pytest.raises(B.DcpError) as e:
        B.dcp_varlen_attn_fwd(q, q, q, cu, 11, False)
    assert e.value.code == B.DCP_ERR_INVALID_ARG


def test_launch_counter_and_profile():
    w = inputs.config(1, False)
    q, k, v, g = inputs.make_qkvg(w.total_tokens, w.n_heads, w.head_dim, 4)
    B.dcp_profile_enable(True)
    B.dcp_profile_read()
    before = B.dcp_launch_count()
    run_gpu(q, k, v, g, w.cu_seqlens, False)
    assert B.dcp_launch_count() - before == 4 + 6          # forward: merge + bounds + prep + main; backward: those + 3
    prof = B.dcp_profile_read()
    B.dcp_profile_enable(False)
    assert prof["fwd"][1] == 1 and prof["bwd_main"][1] == 1 and prof["prep"][1] == 2
    assert prof["fwd"][0] > 0 and prof["bwd_main"][0] > 0


def test_host_pipeline_matches_direct_run():
    """Inputs in pinned host memory, results back in host memory, copies overlapped with compute over
    two sets of device buffers: every step must deliver what a direct call on the same inputs gives."""
    from paper_2608_07524_b200.stream import HostPipeline, MicroBatch, StreamRunner
    lengths = [520, 300, 100]                      # planner order: longest first
    cu = np.concatenate([[0], np.cumsum(lengths)]).astype(np.int32)
    T, H, d = int(cu[-1]), 2, 64
    q, k, v, g = inputs.make_qkvg(T, H, d, 50)
    host_in = [x.pin_memory() for x in (q, k, v, g)]
    runners = [StreamRunner(T, len(lengths), H, d, True, "cuda", value_seed=s) for s in (40, 41)]
    pipe = HostPipeline(runners, T)
    mb = MicroBatch(lengths, 0)
    pipe.run(host_in, lambda r: r.run_micro_batch(mb), 5)
    torch.cuda.synchronize()
    for r in runners:
        r.check()
    o, lse, dq, dk, dv = (x.cpu() for x in run_gpu(q, k, v, g, cu, True))
    for s in range(2):
        ho, hdq, hdk, hdv = pipe.host_out[s]
        assert torch.equal(ho, o) and torch.equal(hdk, dk) and torch.equal(hdv, dv)
        assert float((hdq.float() - dq.float()).abs().max()) <= 2e-2
        assert torch.equal(pipe.host_lse[s].view(H, T), lse)


@pytest.mark.parametrize("seed", list(range(12)))
def test_random_length_mixes(seed):
    """Random mixes of empty, tiny, sub-tile, tile-edge and multi-tile sequences: exercises every way
    short runs can be merged and broken up next to sequences that are not merged."""
    rng = np.random.default_rng(1000 + seed)
    pools = [[0], [1, 2, 3, 5, 8, 13], list(range(14, 65)), [63, 64, 65, 66], list(range(67, 128)), [127, 128, 129, 130],
             [200, 256, 257, 300, 511, 640]]
    weights = np.array([1, 6, 3, 2, 2, 2, 1.5])
    n = int(rng.integers(3, 60))
    lengths = [int(rng.choice(pools[int(rng.choice(len(pools), p=weights / weights.sum()))])) for _ in range(n)]
    if sum(lengths) == 0:
        lengths.append(7)
    causal = bool(seed & 1)
    check_full(lengths, int(rng.choice([1, 2, 3])), int(rng.choice([64, 128])), causal, seed=2000 + seed)


@pytest.mark.parametrize("causal", [False, True])
def test_many_sequences_mixed_with_long_ones(causal):
    # more than 1024 sequences (multi-CTA ranking over the merged list) with a few multi-tile ones in between
    rng = np.random.default_rng(77)
    lengths = [int(x) for x in rng.choice([0, 1, 2, 4, 8, 13, 30, 64, 65, 100], size=1300)]
    for pos, L in ((5, 700), (400, 129), (401, 1000), (1299, 300)):
        lengths[pos] = L
    check_full(lengths, 1, 64, causal, seed=78)


@pytest.mark.parametrize("causal", [False, True])
@pytest.mark.parametrize("d", [8, 40, 72, 80, 96, 104, 112, 120])
def test_head_dims_between_the_native_ones(causal, d):
    # head dimensions other than 64 and 128 run zero-padded to the next of the two (72 is the head
    # dimension of the paper's second model: hidden size 1152 over 16 heads)
    check_full([300, 5, 13, 8, 129, 64, 1, 250], 3, d, causal, seed=90 + d)



def test_inconsistent_boundaries_are_reported_not_used():
    """cu_seqlens is device data the host never reads; the work-list kernels check it (starts at 0,
    never decreases, ends at total_tokens, fits the per-tile storage that max_seqlen promised) and, if
    it does not hold, leave an empty work list and a status the host can query.  Outputs stay as
    they were; nothing is read or written out of bounds."""
    dev = "cuda"
    T, H, d = 600, 2, 64
    q, k, v, g = (x.to(dev) for x in inputs.make_qkvg(T, H, d, 60))
    for bad_cu in ([0, 200, 100, 600], [0, 200, 400, 590], [5, 200, 400, 600], [0, 200, 400, 700]):
        cud = torch.tensor(bad_cu, dtype=torch.int32, device=dev)
        ws = B.alloc_workspace(T, 3, H, d, True, dev)
        o = torch.full_like(q, 7.0)
        lse = torch.zeros((H, T), dtype=torch.float32, device=dev)
        B.dcp_varlen_attn_fwd(q, k, v, cud, 300, False, out=o, lse=lse, workspace=ws)
        with pytest.raises(B.DcpError) as e:
            B.dcp_query_status(ws)
        assert e.value.code == B.DCP_ERR_INVALID_ARG
        assert bool((o == 7.0).all())
        dq = torch.full_like(q, 3.0)
        B.dcp_varlen_attn_bwd(q, k, v, o, g, lse, cud, 300, False, dq=dq, dk=torch.empty_like(q), dv=torch.empty_like(q),
                              workspace=ws)
        with pytest.raises(B.DcpError) as e:
            B.dcp_query_status(ws)
        assert e.value.code == B.DCP_ERR_INVALID_ARG and bool((dq == 3.0).all())
        # the same workspace works again with consistent boundaries
        good = torch.tensor([0, 200, 400, 600], dtype=torch.int32, device=dev)
        B.dcp_varlen_attn_fwd(q, k, v, good, 200, False, out=o, lse=lse, workspace=ws)
        B.dcp_query_status(ws)
        assert bool(torch.isfinite(o.float()).all()) and not bool((o == 7.0).all())


@pytest.fixture
def tile_kernels_only():
    B.dcp_set_short_sequence_path(False)
    yield
    B.dcp_set_short_sequence_path(True)


def test_understated_max_seqlen_cannot_overrun_the_workspace(tile_kernels_only):
    # 2000 sequences of 14 tokens declared as "at most 13": none is merged, so the batch has more tiles than
    # the workspace (sized on the promise) holds; the backward must refuse instead of indexing past its storage
    # (on the tile kernels: the short-sequence kernels refuse the forward already, tested above)
    dev = "cuda"
    n, L, H, d = 2000, 14, 1, 64
    T = n * L
    q, k, v, g = (x.to(dev) for x in inputs.make_qkvg(T, H, d, 61))
    cud = torch.arange(0, T + 1, L, dtype=torch.int32, device=dev)
    ws = B.alloc_workspace(T, n, H, d, True, dev)
    o, lse = B.dcp_varlen_attn_fwd(q, k, v, cud, 13, False, workspace=ws)      # forward has no per-tile storage
    B.dcp_query_status(ws)
    dq = torch.full_like(q, 3.0)
    B.dcp_varlen_attn_bwd(q, k, v, o, g, lse, cud, 13, False, dq=dq, dk=torch.empty_like(q), dv=torch.empty_like(q), workspace=ws)
    with pytest.raises(B.DcpError) as e:
        B.dcp_query_status(ws)
    assert e.value.code == B.DCP_ERR_INVALID_ARG and bool((dq == 3.0).all())
    dq, dk, dv = B.dcp_varlen_attn_bwd(q, k, v, o, g, lse, cud, L, False, workspace=ws)      # the truth: fine
    B.dcp_query_status(ws)
    assert bool(torch.isfinite(dq.float()).all())


@pytest.mark.parametrize("causal", [False, True])
def test_merged_by_aligned_windows(causal):
    # no empty sequence and lengths near 64: pairing inside aligned 128-token windows gives fewer tiles
    # than start windows do, so the work-list kernels take their second merging rule
    lengths = [64] * 9 + [60, 4, 64, 32, 32, 33, 31, 64, 200, 64, 64, 50, 14, 64, 1, 63]
    check_full(lengths, 2, 128, causal, seed=95)
    check_full([64] * 40, 1, 64, causal, seed=96)


def test_status_word_is_sticky_and_maps_to_error_codes():
    """The device status word keeps the most severe failure of any call until it is queried; the query
    reports it and clears it.  Codes: 1 or 2 (a kernel gave up a bounded wait / found its shared memory
    misaligned) -> DCP_ERR_TIMEOUT, 3 (inconsistent boundaries) -> DCP_ERR_INVALID_ARG."""
    dev = "cuda"
    T, H, d = 300, 2, 64
    q, k, v, g = (x.to(dev) for x in inputs.make_qkvg(T, H, d, 62))
    ws = B.alloc_workspace(T, 2, H, d, True, dev)
    good = torch.tensor([0, 100, 300], dtype=torch.int32, device=dev)
    bad = torch.tensor([0, 200, 100], dtype=torch.int32, device=dev)
    B.dcp_varlen_attn_fwd(q, k, v, good, 200, False, workspace=ws)
    B.dcp_query_status(ws)                                  # the header is initialised now
    for code, err in ((1, B.DCP_ERR_TIMEOUT), (2, B.DCP_ERR_TIMEOUT), (3, B.DCP_ERR_INVALID_ARG)):
        ws[:4].copy_(torch.tensor([code, 0, 0, 0], dtype=torch.uint8))
        with pytest.raises(B.DcpError) as e:
            B.dcp_query_status(ws)
        assert e.value.code == err
        B.dcp_query_status(ws)                              # cleared by the query
    # a failing call followed by good calls on the same workspace: the failure is still reported
    B.dcp_varlen_attn_fwd(q, k, v, bad, 200, False, workspace=ws)
    o, lse = B.dcp_varlen_attn_fwd(q, k, v, good, 200, False, workspace=ws)
    B.dcp_varlen_attn_bwd(q, k, v, o, g, lse, good, 200, False, workspace=ws)
    with pytest.raises(B.DcpError) as e:
        B.dcp_query_status(ws)
    assert e.value.code == B.DCP_ERR_INVALID_ARG
    B.dcp_query_status(ws)


def test_bounded_wait_gives_up_and_reports_a_timeout():
    """A wait on a barrier nothing arrives at: the kernels' wait helper stops after its poll limit, raises
    the status word and the CTA returns; the context stays usable."""
    dev = "cuda"
    ws = torch.empty(4096, dtype=torch.uint8, device=dev)
    B.dcp_selftest_wait_timeout(ws, 1 << 10)
    with pytest.raises(B.DcpError) as e:
        B.dcp_query_status(ws)
    assert e.value.code == B.DCP_ERR_TIMEOUT
    B.dcp_query_status(ws)
    # the device still works afterwards
    check_full([130, 40], 1, 64, True, seed=63)
    with pytest.raises(B.DcpError):
        B.dcp_selftest_wait_timeout(ws, (1 << 20) + 1)


def test_input_order_work_list_gives_the_same_results():
    # the measurement switch that lists sequences as they come changes the schedule, not the answers
    lengths = [40, 700, 129, 13, 13, 300, 1]
    try:
        B.dcp_set_work_order(True)
        check_full(lengths, 2, 128, True, seed=64)
        check_full([int(x) for x in np.random.default_rng(9).integers(0, 50, size=1200)], 1, 64, False, seed=65)
    finally:
        B.dcp_set_work_order(False)


def test_cta_spans_are_recorded():
    dev = "cuda"
    lengths = [2000, 700, 129]
    cu = np.concatenate([[0], np.cumsum(lengths)]).astype(np.int32)
    q, k, v, g = (x.to(dev) for x in inputs.make_qkvg(int(cu[-1]), 4, 128, 66))
    cud = torch.tensor(cu, device=dev)
    ws = B.alloc_workspace(int(cu[-1]), 3, 4, 128, True, dev)
    o, lse = B.dcp_varlen_attn_fwd(q, k, v, cud, 2000, False, workspace=ws)
    B.dcp_varlen_attn_bwd(q, k, v, o, g, lse, cud, 2000, False, workspace=ws)
    n_sms = torch.cuda.get_device_properties(0).multi_processor_count
    for which in (0, 1):
        begin, end = B.dcp_read_cta_spans(ws, which)
        assert begin.size == min(n_sms, 256) and bool((end >= begin).all()) and bool((begin > 0).all())
        assert int(end.max() - begin.min()) < 10 ** 9          # nanoseconds: well under a second


@pytest.mark.parametrize("lengths", [[300, 5, 13, 129, 64, 700], [13, 1, 0, 7, 16, 9, 12, 3] * 40],
                         ids=["tile kernels", "short-sequence kernels"])
@pytest.mark.parametrize("causal", [False, True])
def test_head_groups_inside_wider_tensors(causal, lengths):
    """The strided entry points run a group of heads in place inside [T, H, d] tensors (the form the head-
    sharded sequence-parallel scheme needs): every group must give, bit for bit, what the plain calls give on
    a contiguous copy of that group, and must leave the other heads' outputs alone."""
    dev = "cuda"
    cu = np.concatenate([[0], np.cumsum(lengths)]).astype(np.int32)
    T, H, d, p = int(cu[-1]), 6, 128, 3
    q, k, v, g = (x.to(dev) for x in inputs.make_qkvg(T, H, d, 97))
    cud = torch.tensor(cu, device=dev)
    o = torch.full_like(q, float("nan"))
    dq, dk, dv = (torch.full_like(q, float("nan")) for _ in range(3))
    Hg = H // p
    for r in range(p):
        hs = slice(r * Hg, (r + 1) * Hg)
        qc, kc, vc, gc = (x[:, hs].contiguous() for x in (q, k, v, g))
        ref_o, ref_lse = B.dcp_varlen_attn_fwd(qc, kc, vc, cud, max(lengths), causal)
        ref_dq, ref_dk, ref_dv = B.dcp_varlen_attn_bwd(qc, kc, vc, ref_o, gc, ref_lse, cud, max(lengths), causal)
        _, lse = B.dcp_varlen_attn_fwd_strided(q[:, hs], k[:, hs], v[:, hs], cud, max(lengths), causal, o[:, hs])
        B.dcp_varlen_attn_bwd_strided(q[:, hs], k[:, hs], v[:, hs], o[:, hs], g[:, hs], lse, cud, max(lengths), causal,
                                      dq[:, hs], dk[:, hs], dv[:, hs])
        torch.cuda.synchronize()
        assert torch.equal(o[:, hs], ref_o) and torch.equal(lse, ref_lse)
        assert torch.equal(dk[:, hs], ref_dk) and torch.equal(dv[:, hs], ref_dv)
        assert float((dq[:, hs].float() - ref_dq.float()).abs().max()) <= 2e-2       # atomics: order may differ
        if r + 1 < p:       # heads of later groups are still untouched
            rest = slice((r + 1) * Hg, H)
            assert bool(torch.isnan(o[:, rest].float()).all()) and bool(torch.isnan(dk[:, rest].float()).all())
    O, L = oracle.attn_fwd(q.cpu(), k.cpu(), v.cpu(), cu, causal)
    rdq, rdk, rdv = oracle.attn_bwd(q.cpu(), k.cpu(), v.cpu(), g.cpu(), cu, causal)
    assert_close("o", o, O)
    assert_close("dq", dq, rdq)
    assert_close("dk", dk, rdk)
    assert_close("dv", dv, rdv)
    # a stride smaller than the group's own width is refused
    rc = B.lib().dcp_varlen_attn_fwd_strided(q.data_ptr(), k.data_ptr(), v.data_ptr(), cud.data_ptr(), len(lengths), T,
                                             max(lengths), Hg, d, Hg * d - 8, 0, 0.0, o.data_ptr(), lse.data_ptr(),
                                             B.alloc_workspace(T, len(lengths), Hg, d, False, dev).data_ptr(), 1 << 20, None)
    assert rc == B.DCP_ERR_INVALID_ARG
