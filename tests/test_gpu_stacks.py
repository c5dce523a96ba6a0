"""Per-layer parity of the two model-shaped stacks, in the layout and path selection the benchmark uses
(bf16, NHWC, automatic path): YOLOv5s-shaped layers in full at batch 1, RetinaNet-R50-FPN-shaped layers at
the benchmark's batch 4 on sampled outputs (corners included)."""
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


def test_retinanet_stack_unique_layers_batch4_sampled():
    masks = orc.pattern_preset(4, orc.PRESET_CENTRE8)
    rng = np.random.default_rng(11)
    N = 4
    for i, L in enumerate(_unique(synth.retinanet_r50fpn_stack())):
        ks, s, Cin, Cout, H, W = L["ksize"], L["stride"], L["cin"], L["cout"], L["H"], L["W"]
        x = synth.round_like(synth.activations(41, 600 + i, N, Cin, H, W), "bf16")
        w = synth.kaiming_weights(41, 600 + i, Cout, Cin, ks)
        b = synth.bias(41, 600 + i, Cout)
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
