"""GPU parity of the glue kernels (max-pooling, 2x up-sampling, add + activation) against the CPU oracle:
bit-exact (pooling and up-sampling move values; the sum is formed in fp32 and rounded once, and fp32 holds
the sum of two 16-bit values exactly)."""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu

if torch.cuda.is_available():
    from oracle import rtoss_oracle as orc
    from paper_2303_02191_b200 import binding as rt
    from paper_2303_02191_b200 import synth
    import gpu_util as gu


@pytest.mark.parametrize("layout", ["nchw", "nhwc"])
@pytest.mark.parametrize("dt", ["bf16", "f32"])
def test_maxpool_and_upsample(layout, dt):
    lay = rt.NHWC if layout == "nhwc" else rt.NCHW
    N, C, H, W = 2, 24, 13, 10
    x = synth.round_like(synth.activations(61, 1, N, C, H, W), dt)
    xd = gu.to_dev(x, dt, layout)
    for k, s, p in ((5, 1, 2), (3, 2, 1), (2, 2, 0)):
        Ho, Wo = (H + 2 * p - k) // s + 1, (W + 2 * p - k) // s + 1
        Cs, off = C + 8, 5
        shape = (N, Ho, Wo, Cs) if layout == "nhwc" else (N, Cs, Ho, Wo)
        yd = torch.full(shape, 7.0, dtype=gu.TORCH_DT[dt], device="cuda")
        rt.rtoss_maxpool2d(xd, yd, N, C, H, W, k, s, p, lay, off, Cs)
        y = gu.from_dev(yd, layout)
        assert np.array_equal(y[:, off:off + C], orc.maxpool2d(x, k, s, p))
        assert (y[:, :off] == 7.0).all() and (y[:, off + C:] == 7.0).all()
    shape = (N, 2 * H, 2 * W, C) if layout == "nhwc" else (N, C, 2 * H, 2 * W)
    yd = torch.empty(shape, dtype=gu.TORCH_DT[dt], device="cuda")
    rt.rtoss_upsample2x(xd, yd, N, C, H, W, lay)
    assert np.array_equal(gu.from_dev(yd, layout), orc.upsample2x(x))


@pytest.mark.parametrize("dt", ["bf16", "f16", "f32"])
def test_add_act(dt):
    a = synth.round_like(synth.activations(62, 1, 1, 7, 33, 5), dt)
    b = synth.round_like(synth.activations(62, 2, 1, 7, 33, 5), dt)
    ad, bd = gu.to_dev(a, dt), gu.to_dev(b, dt)
    for act, code in (("none", rt.ACT_NONE), ("relu", rt.ACT_RELU)):
        yd = torch.empty_like(ad)
        rt.rtoss_add_act(ad, bd, yd, code)
        ref = orc.add_act(a, b, {"none": orc.ACT_NONE, "relu": orc.ACT_RELU}[act], gu.ORC_DT[dt])
        got = gu.from_dev(yd)
        if dt == "f32":
            assert np.abs(got - ref).max() <= 1e-6 * max(1.0, np.abs(ref).max())
        else:
            assert np.array_equal(got, ref)
    with pytest.raises(rt.RtossError):
        rt.rtoss_maxpool2d(ad, bd, 1, 7, 33, 5, 3, 1, 2)       # padding wider than half the window


@pytest.mark.parametrize("dt", ["bf16", "f16"])
def test_vectorised_nhwc_paths(dt):
    """16-bit NHWC tensors with channel counts and slices in multiples of eight take the 16-byte kernels:
    the same bits as the oracle, neighbours of the written slice untouched."""
    N, C, H, W = 2, 24, 13, 10
    x = synth.round_like(synth.activations(63, 1, N, C, H, W), dt)
    xd = gu.to_dev(x, dt, "nhwc")
    Cs, off = C + 16, 8
    for k, s, p in ((5, 1, 2), (3, 2, 1), (1, 1, 0)):
        Ho, Wo = (H + 2 * p - k) // s + 1, (W + 2 * p - k) // s + 1
        yd = torch.full((N, Ho, Wo, Cs), 7.0, dtype=gu.TORCH_DT[dt], device="cuda")
        rt.rtoss_maxpool2d(xd, yd, N, C, H, W, k, s, p, rt.NHWC, off, Cs)
        y = gu.from_dev(yd, "nhwc")
        assert np.array_equal(y[:, off:off + C], orc.maxpool2d(x, k, s, p))
        assert (y[:, :off] == 7.0).all() and (y[:, off + C:] == 7.0).all()
    yd = torch.full((N, 2 * H, 2 * W, Cs), 7.0, dtype=gu.TORCH_DT[dt], device="cuda")
    rt.rtoss_upsample2x(xd, yd, N, C, H, W, rt.NHWC, off, Cs)
    y = gu.from_dev(yd, "nhwc")
    assert np.array_equal(y[:, off:off + C], orc.upsample2x(x))
    assert (y[:, :off] == 7.0).all() and (y[:, off + C:] == 7.0).all()
    b = synth.round_like(synth.activations(63, 2, N, C, H, W), dt)
    bd = gu.to_dev(b, dt, "nhwc")
    for act, code in (("none", rt.ACT_NONE), ("relu", rt.ACT_RELU)):
        od = torch.empty_like(xd)
        rt.rtoss_add_act(xd, bd, od, code)
        ref = orc.add_act(x, b, {"none": orc.ACT_NONE, "relu": orc.ACT_RELU}[act], gu.ORC_DT[dt])
        assert np.array_equal(gu.from_dev(od, "nhwc"), ref)
