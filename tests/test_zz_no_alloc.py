"""The no-allocation forward entry point gives the same result as the regular one.

Some callers of this library may not allocate device memory at the moment they need attention (a
memory-pool callback, a real-time loop, a host program that hands a plug-in fixed buffers).  For
them dcp_varlen_attn_fwd_noalloc keeps its work-list scratch in a fixed array inside the library.
This file runs last (its name sorts after every other test file) so that a failure here cannot hide
the results of the other tests; it must also pass when run alone in a fresh process.
"""
import numpy as np
import pytest
import torch

from paper_2608_07524_b200 import binding as B
from paper_2608_07524_b200 import inputs

pytestmark = pytest.mark.gpu


def _regular(q, k, v, cu, max_len, causal):
    ws = B.alloc_workspace(q.shape[0], cu.numel() - 1, q.shape[1], q.shape[2], False, q.device)
    o, lse = B.dcp_varlen_attn_fwd(q, k, v, cu, max_len, causal, workspace=ws)
    B.dcp_query_status(ws)
    return o, lse


@pytest.mark.parametrize("causal", [False, True])
def test_two_calls_in_a_row_match_the_regular_entry_point(causal):
    dev = "cuda"
    # two different batches back to back: the second call finds the first call's work list in the
    # shared scratch and must not be affected by it
    batches = [([300, 1000, 129, 128, 1, 513], 3, 128, 31), ([17, 64, 100, 255, 700], 2, 64, 32)]
    for lengths, H, d, seed in batches:
        cu_host = np.concatenate([[0], np.cumsum(lengths)]).astype(np.int32)
        q, k, v, _ = (x.to(dev) for x in inputs.make_qkvg(int(cu_host[-1]), H, d, seed))
        cu = torch.tensor(cu_host, device=dev)
        ref_o, ref_lse = _regular(q, k, v, cu, max(lengths), causal)
        out = torch.full_like(q, float("nan"))
        lse = torch.full((H, q.shape[0]), float("nan"), dtype=torch.float32, device=dev)
        B.dcp_varlen_attn_fwd_noalloc(q, k, v, cu, max(lengths), causal, out, lse)
        B.dcp_noalloc_status()
        # same kernels, same inputs: within the tolerance the parity tests use (in fact identical)
        diff = (out.double() - ref_o.double()).abs()
        rel = float(torch.linalg.norm(out.double() - ref_o.double()) / torch.linalg.norm(ref_o.double()))
        assert float(diff.max()) <= 5e-2 and rel <= 1e-2
        assert float((lse.double() - ref_lse.double()).abs().max()) <= 2e-3
        assert bool(torch.isfinite(out.float()).all()) and bool(torch.isfinite(lse).all())


def test_rejects_more_sequences_than_the_built_in_scratch_holds():
    dev = "cuda"
    n = B.NOALLOC_MAX_SEQS + 1
    q = torch.zeros((n, 1, 64), dtype=torch.bfloat16, device=dev)
    cu = torch.arange(n + 1, dtype=torch.int32, device=dev)
    out = torch.zeros_like(q)
    lse = torch.zeros((1, n), dtype=torch.float32, device=dev)
    with pytest.raises(B.DcpError) as e:
        B.dcp_varlen_attn_fwd_noalloc(q, q, q, cu, 1, False, out, lse)
    assert e.value.code == B.DCP_ERR_UNSUPPORTED
    assert "4096" in str(e.value)


def test_matches_the_oracle_including_short_sequences():
    # the oracle directly (not only the regular entry point), on a batch the regular path would merge into
    # shared tiles and this one runs sequence by sequence
    import oracle
    dev = "cuda"
    lengths = [5, 13, 1, 64, 0, 130, 8, 8, 8, 300, 2]
    cu_host = np.concatenate([[0], np.cumsum(lengths)]).astype(np.int32)
    q, k, v, _ = inputs.make_qkvg(int(cu_host[-1]), 2, 64, 33)
    for causal in (False, True):
        out = torch.full(q.shape, float("nan"), dtype=torch.bfloat16, device=dev)
        lse = torch.full((2, q.shape[0]), float("nan"), dtype=torch.float32, device=dev)
        B.dcp_varlen_attn_fwd_noalloc(q.to(dev), k.to(dev), v.to(dev), torch.tensor(cu_host, device=dev), max(lengths),
                                      causal, out, lse)
        B.dcp_noalloc_status()
        O, L = oracle.attn_fwd(q, k, v, cu_host, causal)
        got = out.double().cpu().numpy()
        assert float(np.max(np.abs(got - O))) <= 5e-2 and float(np.linalg.norm(got - O) / np.linalg.norm(O)) <= 1e-2
        assert float(np.max(np.abs(lse.double().cpu().numpy() - L))) <= 2e-3


def test_thousands_of_sequences_and_no_device_allocation():
    # above 1024 sequences the work list is ranked by a separate kernel; the accepted range goes to 4096
    dev = "cuda"
    rng = np.random.default_rng(34)
    lengths = [int(x) for x in rng.choice([0, 1, 3, 13, 40, 64, 65, 129, 300], size=3000)]
    lengths[17], lengths[2999] = 900, 257
    cu_host = np.concatenate([[0], np.cumsum(lengths)]).astype(np.int32)
    q, k, v, _ = (x.to(dev) for x in inputs.make_qkvg(int(cu_host[-1]), 1, 64, 35))
    cu = torch.tensor(cu_host, device=dev)
    ref_o, ref_lse = _regular(q, k, v, cu, max(lengths), True)
    out = torch.full_like(q, float("nan"))
    lse = torch.full((1, q.shape[0]), float("nan"), dtype=torch.float32, device=dev)
    B.dcp_varlen_attn_fwd_noalloc(q, k, v, cu, max(lengths), True, out, lse)       # first call: address look-up done
    torch.cuda.synchronize()
    free0, alloc0, reserved0 = torch.cuda.mem_get_info()[0], torch.cuda.memory_allocated(), torch.cuda.memory_reserved()
    B.dcp_varlen_attn_fwd_noalloc(q, k, v, cu, max(lengths), True, out, lse)
    B.dcp_noalloc_status()
    # neither the library nor the wrapper took device memory for the call
    assert torch.cuda.mem_get_info()[0] == free0
    assert torch.cuda.memory_allocated() == alloc0 and torch.cuda.memory_reserved() == reserved0
    assert float((out.double() - ref_o.double()).abs().max()) <= 5e-2
    assert float(torch.linalg.norm(out.double() - ref_o.double()) / torch.linalg.norm(ref_o.double())) <= 1e-2
    assert float((lse.double() - ref_lse.double()).abs().max()) <= 2e-3


def test_inconsistent_boundaries_leave_outputs_alone_and_are_reported():
    dev = "cuda"
    q, k, v, _ = (x.to(dev) for x in inputs.make_qkvg(600, 2, 64, 36))
    out = torch.full_like(q, float("nan"))
    lse = torch.full((2, 600), float("nan"), dtype=torch.float32, device=dev)
    bad = torch.tensor([0, 200, 100, 600], dtype=torch.int32, device=dev)
    B.dcp_varlen_attn_fwd_noalloc(q, k, v, bad, 300, False, out, lse)
    with pytest.raises(B.DcpError) as e:
        B.dcp_noalloc_status()
    assert e.value.code == B.DCP_ERR_INVALID_ARG
    assert bool(torch.isnan(out.float()).all()) and bool(torch.isnan(lse).all())
    good = torch.tensor([0, 200, 400, 600], dtype=torch.int32, device=dev)
    B.dcp_varlen_attn_fwd_noalloc(q, k, v, good, 200, False, out, lse)
    B.dcp_noalloc_status()
    assert bool(torch.isfinite(out.float()).all()) and bool(torch.isfinite(lse).all())
