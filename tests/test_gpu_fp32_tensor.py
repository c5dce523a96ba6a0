"""fp32 on the tensor path: kind::tf32 instructions with every value split into a tf32 head and its remainder, three
products per tap (head x head, head x remainder, remainder x head) accumulated in fp32.  The bound is the fp32 one,
1e-4 of max(|ref|, rms(ref)), against the CPU oracle (double accumulation), NHWC, through the C ABI."""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu

if torch.cuda.is_available():
    from oracle import rtoss_oracle as orc
    from paper_2303_02191_b200 import binding as rt
    from paper_2303_02191_b200 import synth
    import gpu_util as gu


def _table(k):
    preset = {2: orc.PRESET_CONN4, 3: orc.PRESET_CONN4, 4: orc.PRESET_CENTRE8, 9: orc.PRESET_DENSE}[k]
    return orc.pattern_preset(k, preset)


CASES = [
    # ksize, N, Cin, Cout, H, W, stride, k, act
    (3, 1, 32, 32, 32, 32, 1, 4, "none"),       # the 32-channel test layer
    (3, 1, 32, 32, 32, 32, 1, 4, "silu"),
    (3, 2, 64, 64, 20, 20, 1, 2, "silu"),       # narrow layer: filters repeated down the rows
    (3, 1, 256, 256, 20, 20, 1, 4, "silu"),     # eight channel blocks of 32, two filter tiles
    (3, 1, 256, 256, 40, 40, 1, 9, "relu"),     # dense table
    (3, 1, 36, 200, 13, 17, 1, 3, "none"),      # ragged channel block (4 channels in the last), ragged filter tile
    (3, 1, 64, 128, 40, 40, 2, 4, "silu"),      # stride 2: four staged sub-tiles per block
    (3, 1, 512, 512, 7, 9, 1, 4, "relu"),       # few tiles, sixteen channel blocks: cut along K through a cluster
    (1, 2, 256, 128, 40, 40, 1, 3, "silu"),     # 1x1 with left-over weights
    (1, 1, 64, 32, 20, 20, 1, 4, "relu"),       # few filters (fp32 keeps the filters on M)
    (1, 1, 128, 256, 25, 34, 2, 4, "none"),     # 1x1 stride 2
]


@pytest.mark.parametrize("ks,N,Cin,Cout,H,W,stride,k,act", CASES)
def test_fp32_tensor_path_against_the_oracle(ks, N, Cin, Cout, H, W, stride, k, act):
    err = gu.check_layer(81, ks * 1000 + Cin + Cout + H, ks, N, Cin, Cout, H, W, stride, k, _table(k), "f32", act, "nhwc",
                         path=rt.PATH_TENSOR)
    assert err <= 1e-4
    assert gu.ctx().rtoss_device_status() == 0


def test_fp32_residual_slice_and_group():
    c = gu.ctx()
    masks = _table(4)
    # residual in front of the activation, output written into a channel slice of a wider tensor
    N, Cin, Cout, H, W = 1, 64, 128, 16, 16
    x = synth.activations(82, 1, N, Cin, H, W)
    w = synth.kaiming_weights(82, 1, Cout, Cin, 3)
    b = synth.bias(82, 1, Cout)
    res = synth.activations(82, 2, N, 160, H, W)
    pid_g, packed = gu.select_pack(w, 3, masks, 4, "f32")
    _, wd, _ = gu.oracle_weights(w, 3, masks, 4, "f32")
    xd, bd = gu.to_dev(x, "f32", "nhwc"), torch.from_numpy(b).cuda()
    rd = gu.to_dev(res, "f32", "nhwc")
    yd = torch.full((N, H, W, 160), 7.0, device="cuda")
    c.rtoss_conv3x3_pattern(packed, xd, yd, N, H, W, 1, rt.NHWC, rt.ACT_RELU, bd, 32, 160, rt.PATH_TENSOR, residual=rd)
    torch.cuda.synchronize()
    y = gu.from_dev(yd, "nhwc")
    ref = orc.add_act(orc.conv3x3(x, wd, b, 1, orc.ACT_NONE, orc.DT_F32), res[:, 32:160], orc.ACT_RELU, orc.DT_F32)
    assert orc.rel_err(y[:, 32:160], ref) <= 1e-4
    assert np.all(y[:, :32] == 7.0)
    # three fp32 convolutions in one launch (one weight tensor over three sizes)
    items, outs = [], []
    for i, (h, w_) in enumerate([(30, 40), (15, 20), (8, 10)]):
        xi = synth.activations(82, 10 + i, 2, Cin, h, w_)
        xid = gu.to_dev(xi, "f32", "nhwc")
        yid = torch.zeros(2, h, w_, Cout, device="cuda")
        items.append(c.conv_item(packed, xid, yid, 2, h, w_, 1, rt.NHWC, rt.ACT_SILU, bd))
        outs.append((xi, xid, yid))
    assert c.rtoss_conv_group(items) == 1
    torch.cuda.synchronize()
    for xi, _, yid in outs:
        ref = orc.conv3x3(xi, wd, b, 1, orc.ACT_SILU, orc.DT_F32)
        assert orc.rel_err(gu.from_dev(yid, "nhwc"), ref) <= 1e-4
    packed.close()
    assert c.rtoss_device_status() == 0


def test_fp32_large_point_sampled():
    """C = 256, 80 x 80, batch 4 on sampled outputs: many tiles per CTA."""
    rng = np.random.default_rng(14)
    masks = _table(4)
    N, C, HW = 4, 256, 80
    w = synth.kaiming_weights(83, 1, C, C, 3)
    b = synth.bias(83, 1, C)
    x = synth.activations(83, 1, N, C, HW, HW)
    pid_g, packed = gu.select_pack(w, 3, masks, 4, "f32")
    pid_o, wd, _ = gu.oracle_weights(w, 3, masks, 4, "f32")
    assert np.array_equal(pid_g, pid_o.ravel())
    y = gu.run_conv(packed, 3, x, "f32", 1, "silu", b, "nhwc", path=rt.PATH_TENSOR)
    npts = 3000
    idx = np.stack([rng.integers(0, N, npts), rng.integers(0, C, npts), rng.integers(0, HW, npts), rng.integers(0, HW, npts)],
                   axis=1).astype(np.int32)
    idx[:3] = [[0, 0, 0, 0], [N - 1, C - 1, HW - 1, HW - 1], [0, C - 1, 0, HW - 1]]
    ref = orc.conv_points(3, x, wd, b, 1, orc.ACT_SILU, orc.DT_F32, idx)
    got = y[idx[:, 0], idx[:, 1], idx[:, 2], idx[:, 3]]
    rms = float(np.sqrt(np.mean(ref.astype(np.float64) ** 2)))
    assert np.max(np.abs(got - ref) / np.maximum(np.abs(ref), rms)) <= 1e-4
    packed.close()
    assert gu.ctx().rtoss_device_status() == 0
