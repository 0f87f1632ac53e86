"""The workload generator reproduces the stored length lists and the SplitMix64 test vector."""
import os

from paper_2608_07524_b200 import inputs

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def read_ints(name, base=10):
    with open(os.path.join(GOLD, name)) as f:
        return [int(line, base) for line in f if line.strip() and not line.startswith("#")]


def test_splitmix64_vector():
    g = inputs.SplitMix64(0)
    assert [g.next_u64() for _ in range(3)] == read_ints("splitmix64_seed0.txt", 16)


def test_length_lists():
    assert inputs.text_lengths() == read_ints("lengths_text.txt")
    assert inputs.video_lengths() == read_ints("lengths_video.txt")
    assert inputs.extreme_lengths() == read_ints("lengths_extreme.txt")
    assert sum(inputs.text_lengths()) == 79299
    assert sum(inputs.video_lengths()) == 124992
    assert sum(inputs.extreme_lengths()) == 206646


def test_stream_shape():
    s = inputs.stream_batches()
    assert len(s) == 256 and all(len(b) == 24 for b in s)
    allowed = {256, 1024, 2048, 3328, 1200, 4800, 9600, 15600, 3600, 14400, 28800, 46800}
    assert set(x for b in s for x in b) <= allowed
    assert sum(map(sum, s)) == 34231792


def test_values_are_reproducible_bf16():
    import torch
    a = inputs.make_qkvg(50, 2, 64, 4)
    b = inputs.make_qkvg(50, 2, 64, 4)
    assert all(x.dtype == torch.bfloat16 and torch.equal(x, y) for x, y in zip(a, b))
    assert not torch.equal(a[0], a[1])


def test_flop_convention():
    w = inputs.config(3)
    assert abs(w.fwd_flops() / 1e12 - 22.785) < 0.01 and abs(w.fwd_bwd_flops() / 1e12 - 79.748) < 0.03
    w = inputs.config(2)
    assert abs(w.fwd_bwd_flops() / 1e12 - 4.086) < 0.01


def test_two_dimensional_views_of_the_video_clips():
    clips = inputs.video_clips()
    assert [f * s for f, s in clips] == inputs.video_lengths()
    assert all(inputs.clip_shape(f * s) == (f, s) for f, s in clips)
    spatial, temporal = inputs.short2d_lengths("spatial"), inputs.short2d_lengths("temporal")
    assert sum(spatial) == sum(temporal) == sum(inputs.video_lengths()) == 124992
    assert len(spatial) == sum(f for f, _ in clips) == 121 and set(spatial) == {256, 1200, 3600}
    assert len(temporal) == sum(s for _, s in clips) == 20384 and set(temporal) == {1, 4, 8, 13}
    assert inputs.axis_lengths([(2, 3)], "spatial") == [3, 3] and inputs.axis_lengths([(2, 3)], "temporal") == [2, 2, 2]
    import pytest
    with pytest.raises(ValueError):
        inputs.clip_shape(777)
    with pytest.raises(ValueError):
        inputs.axis_lengths(clips, "diagonal")


def test_cubic_for_exp2_on_the_fma_pipe_is_accurate_enough():
    """The forward kernel evaluates a share of its exponentials as 2^n * p(f), n = round(x), f = x - n in
    [-0.5, 0.5], p a cubic (coefficients as in the kernel), with n added into the exponent field after
    the add-a-magic-number rounding.  Emulated here in fp32: the result must stay well inside the bf16
    rounding (2^-9) that P gets anyway."""
    import numpy as np
    c0, c1, c2, c3 = (np.float32(v) for v in (0.99992807, 0.69326099, 0.24261112, 0.05517162))
    magic = np.float32(12582912.0)
    # arguments reach +8: the running maximum is raised lazily, only once a score exceeds it by 2^8
    x = np.concatenate([np.linspace(-126.0, 8.0, 200001), -np.logspace(-6, 2, 2000)]).astype(np.float32)
    xc = np.maximum(x, np.float32(-126.0))
    t = (xc + magic).astype(np.float32)
    f = (xc - (t - magic).astype(np.float32)).astype(np.float32)
    assert float(np.abs(f).max()) <= 0.5
    q = ((c3 * f + c2) * f + c1) * f + c0
    bits = q.astype(np.float32).view(np.uint32) + (t.view(np.uint32) << np.uint32(23))
    got = bits.view(np.float32).astype(np.float64)
    want = np.exp2(xc.astype(np.float64))
    rel = np.abs(got / want - 1.0)
    assert float(rel.max()) < 1.5e-4 < 2.0 ** -9 / 10
