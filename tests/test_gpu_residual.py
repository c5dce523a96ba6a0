"""Residual operand of the tensor-path convolutions: y = act(round(conv + bias) + residual) in one call.  Checked
against the CPU oracle (convolution without activation, then its element-wise add + activation) and, bit for bit for
act none and ReLU, against the library's own two-call form; on uncut tiles, tiles shared out over a cluster (split K),
the element-store form of ragged filter counts, a channel slice of a wider tensor, stride 2, both 16-bit types, and
with the output aliasing the residual; and the other order, y = round(act(conv + bias)) + residual, bit for bit
against the two-call form for every activation.  Calls the tensor path cannot take must be declined, not computed
elsewhere."""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu

if torch.cuda.is_available():
    from oracle import rtoss_oracle as orc
    from paper_2303_02191_b200 import binding as rt
    from paper_2303_02191_b200 import synth
    import gpu_util as G

CASES = [
    # ksize, Cin, Cout, N, H, W, stride, act, (y_off, y_stride), dtype
    (3, 128, 128, 2, 40, 40, 1, "relu", (0, 0), "bf16"),       # uncut tiles, several per CTA row block, ragged edge
    (3, 128, 128, 1, 23, 31, 1, "none", (0, 0), "bf16"),
    (3, 64, 192, 1, 19, 21, 1, "silu", (0, 0), "bf16"),
    (1, 256, 256, 2, 20, 28, 1, "relu", (0, 0), "bf16"),       # the closing 1x1 of a bottleneck block
    (1, 128, 512, 1, 25, 34, 1, "relu", (0, 0), "f16"),
    (3, 128, 128, 1, 24, 24, 2, "relu", (128, 384), "bf16"),   # stride 2 into a channel slice
    (3, 96, 100, 1, 17, 18, 1, "relu", (0, 0), "bf16"),        # ragged filter count: element stores
    (3, 256, 256, 2, 13, 17, 1, "relu", (0, 0), "bf16"),       # split K over a cluster
    (3, 320, 100, 1, 9, 11, 1, "silu", (0, 0), "bf16"),        # split K, element stores
    (1, 2048, 512, 1, 7, 9, 1, "relu", (0, 0), "bf16"),        # split K, 1x1
    (1, 2048, 256, 1, 10, 10, 1, "none", (0, 0), "f16"),
]


def _setup(ksize, cin, cout, N, H, W, stride, ysl, dt):
    masks = orc.pattern_preset(4, orc.PRESET_CENTRE8)
    w = synth.kaiming_weights(5, 21, cout, cin, ksize)
    b = synth.bias(5, 21, cout)
    x = synth.round_like(synth.activations(5, 21, N, cin, H, W), dt)
    Ho, Wo = synth.out_hw(H, W, stride)
    Cs = ysl[1] if ysl[1] else cout
    res = synth.round_like(synth.activations(5, 22, N, Cs, Ho, Wo), dt)   # a whole tensor shaped like y's buffer
    pid, packed = G.select_pack(w, ksize, masks, 4, dt)
    _, wd, _ = G.oracle_weights(w, ksize, masks, 4, dt)
    return masks, b, x, res, packed, wd, (Ho, Wo, Cs)


@pytest.mark.parametrize("ksize,cin,cout,N,H,W,stride,act,ysl,dt", CASES)
def test_residual_parity(ksize, cin, cout, N, H, W, stride, act, ysl, dt):
    _, b, x, res, packed, wd, (Ho, Wo, Cs) = _setup(ksize, cin, cout, N, H, W, stride, ysl, dt)
    a = {"none": orc.ACT_NONE, "relu": orc.ACT_RELU, "silu": orc.ACT_SILU}[act]
    conv = orc.conv3x3 if ksize == 3 else orc.conv1x1
    plain = conv(x, wd, b, stride, orc.ACT_NONE, G.ORC_DT[dt])
    ref = orc.add_act(plain, res[:, ysl[0]:ysl[0] + cout], a, G.ORC_DT[dt])

    c = G.ctx()
    fn = c.rtoss_conv3x3_pattern if ksize == 3 else c.rtoss_conv1x1_pattern
    xd, bd, rd = G.to_dev(x, dt, "nhwc"), torch.from_numpy(b).cuda(), G.to_dev(res, dt, "nhwc")
    args = (packed, xd, None, N, H, W, stride, rt.NHWC)
    for _ in range(2):
        y = torch.full((N, Ho, Wo, Cs), 7.0, dtype=G.TORCH_DT[dt], device="cuda")
        fn(*args[:2], y, *args[3:], rt.ACT_NAMES[act], bd, ysl[0], ysl[1], rt.PATH_TENSOR, residual=rd)
        torch.cuda.synchronize()
        got = G.from_dev(y, "nhwc")[:, ysl[0]:ysl[0] + cout]
        err = orc.rel_err(got, ref)
        assert err <= G.TOL[dt], "relative error %g" % err
        if ysl[1]:   # channels outside the slice keep what they held
            rest = np.delete(G.from_dev(y, "nhwc"), np.s_[ysl[0]:ysl[0] + cout], axis=1)
            assert np.all(rest == 7.0)

    # the two-call form of the library: same bits for act none and ReLU
    t = torch.zeros((N, Ho, Wo, Cs), dtype=G.TORCH_DT[dt], device="cuda")
    fn(*args[:2], t, *args[3:], rt.ACT_NONE, bd, ysl[0], ysl[1], rt.PATH_TENSOR)
    two = torch.empty_like(t)
    rt.rtoss_add_act(t, rd, two, rt.ACT_NAMES[act])
    torch.cuda.synchronize()
    sl = slice(ysl[0], ysl[0] + cout)
    if act != "silu":
        assert torch.equal(two[..., sl], y[..., sl])
    else:
        assert orc.rel_err(G.from_dev(two, "nhwc")[:, sl], got) <= G.TOL[dt]

    # output aliasing the residual
    y2 = rd.clone()
    fn(*args[:2], y2, *args[3:], rt.ACT_NAMES[act], bd, ysl[0], ysl[1], rt.PATH_TENSOR, residual=y2)
    torch.cuda.synchronize()
    assert torch.equal(y2[..., sl], y[..., sl])
    assert c.rtoss_device_status() == 0
    packed.close()


def test_residual_is_declined_off_the_tensor_path():
    c = G.ctx()
    masks = orc.pattern_preset(4, orc.PRESET_CENTRE8)
    bad = [
        (3, 30, 32, "f32", rt.NHWC),     # 32-bit data whose channel count is no multiple of four (the FMA path takes it)
        (3, 64, 64, "bf16", rt.NCHW),    # planar layout
        (1, 64, 32, "bf16", rt.NHWC),    # narrow 1x1 layer
    ]
    for ksize, cin, cout, dt, lay in bad:
        w = synth.kaiming_weights(5, 23, cout, cin, ksize)
        _, packed = G.select_pack(w, ksize, masks, 4, dt)
        shape = (1, 8, 8, cin) if lay == rt.NHWC else (1, cin, 8, 8)
        oshape = (1, 8, 8, cout) if lay == rt.NHWC else (1, cout, 8, 8)
        x = torch.zeros(shape, dtype=G.TORCH_DT[dt], device="cuda")
        y = torch.full(oshape, 7.0, dtype=G.TORCH_DT[dt], device="cuda")
        r = torch.ones(oshape, dtype=G.TORCH_DT[dt], device="cuda")
        fn = c.rtoss_conv3x3_pattern if ksize == 3 else c.rtoss_conv1x1_pattern
        with pytest.raises(rt.RtossError) as e:
            fn(packed, x, y, 1, 8, 8, 1, lay, rt.ACT_RELU, None, residual=r)
        assert e.value.status == rt.ERR_UNSUPPORTED
        torch.cuda.synchronize()
        assert torch.all(y == 7.0)       # nothing was launched
        packed.close()
    # an unaligned residual pointer
    w = synth.kaiming_weights(5, 23, 128, 128, 3)
    _, packed = G.select_pack(w, 3, masks, 4, "bf16")
    x = torch.zeros((1, 8, 8, 128), dtype=torch.bfloat16, device="cuda")
    y = torch.empty((1, 8, 8, 128), dtype=torch.bfloat16, device="cuda")
    r = torch.zeros(8 * 8 * 128 + 8, dtype=torch.bfloat16, device="cuda")[1:]
    with pytest.raises(rt.RtossError) as e:
        c.rtoss_conv3x3_pattern(packed, x, y, 1, 8, 8, 1, rt.NHWC, rt.ACT_RELU, None, residual=r)
    assert e.value.status == rt.ERR_UNSUPPORTED
    packed.close()


POST_CASES = [
    # ksize, Cin, Cout, N, H, W, stride, act, (y_off, y_stride), dtype: the residual behind the activation
    (3, 32, 32, 2, 40, 40, 1, "silu", (0, 0), "bf16"),         # narrow 3x3: the filters are repeated down the lanes
    (3, 64, 64, 1, 23, 31, 1, "silu", (0, 0), "bf16"),
    (3, 128, 128, 2, 40, 40, 1, "silu", (0, 0), "f16"),
    (3, 128, 128, 1, 24, 24, 2, "relu", (128, 384), "bf16"),
    (3, 256, 256, 1, 13, 17, 1, "silu", (0, 0), "bf16"),       # split K over a cluster
    (3, 320, 100, 1, 9, 11, 1, "silu", (0, 0), "bf16"),        # split K, element stores
    (3, 96, 100, 1, 17, 18, 1, "silu", (0, 0), "bf16"),        # element stores
    (1, 256, 256, 2, 20, 28, 1, "silu", (0, 0), "bf16"),
    (1, 2048, 512, 1, 7, 9, 1, "none", (0, 0), "bf16"),
]


@pytest.mark.parametrize("ksize,cin,cout,N,H,W,stride,act,ysl,dt", POST_CASES)
def test_residual_behind_the_activation(ksize, cin, cout, N, H, W, stride, act, ysl, dt):
    """y = round(act(conv + bias)) + residual: against the oracle (its convolution with the activation, then its add
    without one) and, bit for bit for every activation, against the library's two-call form."""
    _, b, x, res, packed, wd, (Ho, Wo, Cs) = _setup(ksize, cin, cout, N, H, W, stride, ysl, dt)
    a = {"none": orc.ACT_NONE, "relu": orc.ACT_RELU, "silu": orc.ACT_SILU}[act]
    conv = orc.conv3x3 if ksize == 3 else orc.conv1x1
    ref = orc.add_act(conv(x, wd, b, stride, a, G.ORC_DT[dt]), res[:, ysl[0]:ysl[0] + cout], orc.ACT_NONE, G.ORC_DT[dt])
    c = G.ctx()
    fn = c.rtoss_conv3x3_pattern if ksize == 3 else c.rtoss_conv1x1_pattern
    xd, bd, rd = G.to_dev(x, dt, "nhwc"), torch.from_numpy(b).cuda(), G.to_dev(res, dt, "nhwc")
    sl = slice(ysl[0], ysl[0] + cout)
    y = torch.full((N, Ho, Wo, Cs), 7.0, dtype=G.TORCH_DT[dt], device="cuda")
    fn(packed, xd, y, N, H, W, stride, rt.NHWC, rt.ACT_NAMES[act], bd, ysl[0], ysl[1], rt.PATH_TENSOR, residual=rd,
       residual_after_act=True)
    torch.cuda.synchronize()
    err = orc.rel_err(G.from_dev(y, "nhwc")[:, sl], ref)
    assert err <= G.TOL[dt], "relative error %g" % err
    t = torch.zeros((N, Ho, Wo, Cs), dtype=G.TORCH_DT[dt], device="cuda")
    fn(packed, xd, t, N, H, W, stride, rt.NHWC, rt.ACT_NAMES[act], bd, ysl[0], ysl[1], rt.PATH_TENSOR)
    two = torch.empty_like(t)
    rt.rtoss_add_act(t, rd, two, rt.ACT_NONE)
    torch.cuda.synchronize()
    assert torch.equal(two[..., sl], y[..., sl])
    assert c.rtoss_device_status() == 0
    packed.close()
