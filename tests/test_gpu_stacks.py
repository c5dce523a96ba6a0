"""Per-layer parity of the two model-shaped stacks, in the layout and path selection the benchmark uses
(bf16, NHWC, automatic path): YOLOv5s-shaped layers in full at batch 1 and on sampled outputs at the benchmark's
batch 16, RetinaNet-R50-FPN-shaped layers at the benchmark's batch 4 on sampled outputs (corners included)."""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu

if torch.cuda.is_available():
    from oracle import rtoss_oracle as orc
    from paper_2303_02191_b200 import binding as rt
    from paper_2303_02191_b200 import synth
    import gpu_util as gu

ACT = {"none": 0, "relu": 1, "silu": 2}


def _unique(layers):
    seen, out = set(), []
    for L in layers:
        key = (L["ksize"], L["stride"], L["cin"], L["cout"], L["H"], L["W"], L["act"])
        if key not in seen:
            seen.add(key)
            out.append(L)
    return out


def test_yolov5s_stack_every_unique_layer_full_tensor():
    masks = orc.pattern_preset(4, orc.PRESET_CENTRE8)
    worst = 0.0
    for i, L in enumerate(_unique(synth.yolov5s_stack())):
        err = gu.check_layer(40, 500 + i, L["ksize"], 1, L["cin"], L["cout"], L["H"], L["W"], L["stride"], 4, masks, "bf16",
                             L["act"], "nhwc")
        worst = max(worst, err)
    assert gu.ctx().rtoss_device_status() == 0
    assert worst <= 2e-2


def _sampled_stack(layers, N, seed, tid0, rng):
    masks = orc.pattern_preset(4, orc.PRESET_CENTRE8)
    for i, L in enumerate(_unique(layers)):
        ks, s, Cin, Cout, H, W = L["ksize"], L["stride"], L["cin"], L["cout"], L["H"], L["W"]
        x = synth.round_like(synth.activations(seed, tid0 + i, N, Cin, H, W), "bf16")
        w = synth.kaiming_weights(seed, tid0 + i, Cout, Cin, ks)
        b = synth.bias(seed, tid0 + i, Cout)
        pid_g, packed = gu.select_pack(w, ks, masks, 4, "bf16")
        pid_o, wd, _ = gu.oracle_weights(w, ks, masks, 4, "bf16")
        assert np.array_equal(pid_g, pid_o.ravel()), L["name"]
        y = gu.run_conv(packed, ks, x, "bf16", s, L["act"], b, "nhwc")
        Ho, Wo = synth.out_hw(H, W, s)
        npts = 1500
        idx = np.stack([rng.integers(0, N, npts), rng.integers(0, Cout, npts), rng.integers(0, Ho, npts),
                        rng.integers(0, Wo, npts)], axis=1).astype(np.int32)
        idx[:4] = [[0, 0, 0, 0], [0, 0, 0, Wo - 1], [N - 1, Cout - 1, Ho - 1, Wo - 1], [N - 1, 0, Ho - 1, 0]]
        ref = orc.conv_points(ks, x, wd, b, s, ACT[L["act"]], orc.DT_BF16, idx)
        got = y[idx[:, 0], idx[:, 1], idx[:, 2], idx[:, 3]]
        rms = float(np.sqrt(np.mean(ref.astype(np.float64) ** 2)))
        err = np.max(np.abs(got - ref) / np.maximum(np.abs(ref), max(rms, 1e-30)))
        assert err <= 2e-2, (L["name"], err)
        assert np.isfinite(y).all()
        packed.close()
        del x, y
    assert gu.ctx().rtoss_device_status() == 0


def test_retinanet_stack_unique_layers_batch4_sampled():
    _sampled_stack(synth.retinanet_r50fpn_stack(), 4, 41, 600, np.random.default_rng(11))


def test_yolov5s_stack_unique_layers_batch16_sampled():
    """The batch the benchmark times: the tile walk over sixteen images of every layer shape of the stack."""
    _sampled_stack(synth.yolov5s_stack(), 16, 44, 700, np.random.default_rng(13))


SWEEP_SUBSET = [(dt, C, HW, k) for dt in ("bf16", "f32") for C in (64, 256) for HW in (20, 40) for k in (2, 3, 4, 9)]


@pytest.mark.parametrize("dt,C,HW,k", SWEEP_SUBSET, ids=lambda v: str(v))
def test_sweep_points_batch1_full_tensor(dt, C, HW, k):
    """Points of the isolated-3x3 sweep the oracle finishes quickly, in the sweep's own launch configuration:
    bf16 NHWC (automatic path) and fp32 NCHW."""
    preset = {2: orc.PRESET_CONN4, 3: orc.PRESET_CONN4, 4: orc.PRESET_CENTRE8, 9: orc.PRESET_DENSE}[k]
    masks = orc.pattern_preset(k, preset)
    gu.check_layer(42, 800 + C + HW + k, 3, 1, C, C, HW, HW, 1, k, masks, dt, "silu", "nhwc" if dt == "bf16" else "nchw")


def test_sweep_large_point_sampled():
    """The largest point of the sweep (C = 512, 160 x 160, batch 32 is cut to batch 2 to bound memory and time)
    on sampled outputs, both dtypes."""
    rng = np.random.default_rng(12)
    masks = orc.pattern_preset(4, orc.PRESET_CENTRE8)
    N, C, HW = 2, 512, 160
    w = synth.kaiming_weights(43, 1, C, C, 3)
    b = synth.bias(43, 1, C)
    for dt, layout in (("bf16", "nhwc"), ("f32", "nchw")):
        x = synth.round_like(synth.activations(43, 1, N, C, HW, HW), dt)
        pid_g, packed = gu.select_pack(w, 3, masks, 4, dt)
        pid_o, wd, _ = gu.oracle_weights(w, 3, masks, 4, dt)
        assert np.array_equal(pid_g, pid_o.ravel())
        y = gu.run_conv(packed, 3, x, dt, 1, "silu", b, layout)
        npts = 2000
        idx = np.stack([rng.integers(0, N, npts), rng.integers(0, C, npts), rng.integers(0, HW, npts),
                        rng.integers(0, HW, npts)], axis=1).astype(np.int32)
        idx[:3] = [[0, 0, 0, 0], [N - 1, C - 1, HW - 1, HW - 1], [0, C - 1, 0, HW - 1]]
        ref = orc.conv_points(3, x, wd, b, 1, orc.ACT_SILU, gu.ORC_DT[dt], idx)
        got = y[idx[:, 0], idx[:, 1], idx[:, 2], idx[:, 3]]
        rms = float(np.sqrt(np.mean(ref.astype(np.float64) ** 2)))
        assert np.max(np.abs(got - ref) / np.maximum(np.abs(ref), rms)) <= gu.TOL[dt]
        packed.close()
    assert gu.ctx().rtoss_device_status() == 0
