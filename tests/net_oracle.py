"""The YOLOv5s-shaped program of `paper_2303_02191_b200.yolov5s_net` executed by the CPU oracle (test side)."""
import numpy as np

from paper_2303_02191_b200 import synth
from paper_2303_02191_b200.yolov5s_net import OUTPUTS, program


def oracle_forward(x_nchw, H0, W0, k=4, seed=0, dtype="bf16"):
    """The same program in the CPU oracle (NCHW float arrays holding values rounded to `dtype`)."""
    from oracle import rtoss_oracle as orc
    odt = {"bf16": orc.DT_BF16, "f16": orc.DT_F16}[dtype]
    ops, bufs, layers = program(H0, W0)
    N = x_nchw.shape[0]
    t = {n: np.zeros((N, C, H, W), dtype=np.float32) for n, (C, H, W) in bufs.items()}
    t["in"] = synth.round_like(x_nchw, dtype)
    masks = orc.pattern_preset(k, orc.PRESET_CENTRE8 if k == 4 else orc.PRESET_CONN4)
    for op in ops:
        if op[0] == "conv":
            _, i, src, dst, off = op
            L = layers[i]
            w = synth.kaiming_weights(seed, 2000 + i, L["cout"], L["cin"], L["ksize"])
            b = synth.bias(seed, 2000 + i, L["cout"])
            if L["ksize"] == 3:
                pid = orc.select_3x3(w, masks)
                wd = orc.unpack_3x3(orc.pack_3x3(w, masks, k, pid, odt)[0], L["cout"], L["cin"], masks, k, pid)
                y = orc.conv3x3(t[src], wd, b, L["stride"], orc.ACT_SILU, odt)
            else:
                w2 = w.reshape(L["cout"], L["cin"])
                pid = orc.select_1x1(w2, masks)
                wd = orc.unpack_1x1(orc.pack_1x1(w2, masks, k, pid, odt), L["cout"], L["cin"], masks, k, pid)
                y = orc.conv1x1(t[src], wd, b, L["stride"], orc.ACT_SILU, odt)
            t[dst][:, off:off + L["cout"]] = y
        elif op[0] == "add":
            t[op[3]] = orc.add_act(t[op[1]], t[op[2]], orc.ACT_NONE, odt)
        elif op[0] == "pool5":
            C = bufs[op[1]][0]
            t[op[2]][:, op[3]:op[3] + C] = orc.maxpool2d(t[op[1]], 5, 1, 2)
        elif op[0] == "up":
            C = bufs[op[1]][0]
            t[op[2]][:, op[3]:op[3] + C] = orc.upsample2x(t[op[1]])
        elif op[0] == "copy":
            C = bufs[op[1]][0]
            t[op[2]][:, op[3]:op[3] + C] = t[op[1]]
    return {n: t[n] for n in OUTPUTS}


def oracle_forward_retinanet(x_nchw, H0, W0, k=4, seed=0, dtype="bf16"):
    """The RetinaNet-shaped program of `paper_2303_02191_b200.retinanet_net` in the CPU oracle; x is the
    64-channel tensor behind the stem, N x 64 x H0/4 x W0/4."""
    from oracle import rtoss_oracle as orc
    from paper_2303_02191_b200 import retinanet_net
    odt = {"bf16": orc.DT_BF16, "f16": orc.DT_F16}[dtype]
    acts = {"none": orc.ACT_NONE, "relu": orc.ACT_RELU, "silu": orc.ACT_SILU}
    ops, bufs, layers, outputs = retinanet_net.program(H0, W0)
    t = {"in": synth.round_like(x_nchw, dtype)}
    masks = orc.pattern_preset(k, orc.PRESET_CENTRE8 if k == 4 else orc.PRESET_CONN4)
    dense = {}
    for op in ops:
        if op[0] == "conv":
            _, i, src, dst, act = op
            L = layers[i]
            if L["wid"] not in dense:
                w = synth.kaiming_weights(seed, 3000 + L["wid"], L["cout"], L["cin"], L["ksize"])
                b = synth.bias(seed, 3000 + L["wid"], L["cout"])
                if L["ksize"] == 3:
                    pid = orc.select_3x3(w, masks)
                    wd = orc.unpack_3x3(orc.pack_3x3(w, masks, k, pid, odt)[0], L["cout"], L["cin"], masks, k, pid)
                else:
                    w2 = w.reshape(L["cout"], L["cin"])
                    pid = orc.select_1x1(w2, masks)
                    wd = orc.unpack_1x1(orc.pack_1x1(w2, masks, k, pid, odt), L["cout"], L["cin"], masks, k, pid)
                dense[L["wid"]] = (wd, b)
            wd, b = dense[L["wid"]]
            fn = orc.conv3x3 if L["ksize"] == 3 else orc.conv1x1
            t[dst] = fn(t[src], wd, b, L["stride"], acts[act], odt)
        elif op[0] == "add":
            t[op[3]] = orc.add_act(t[op[1]], t[op[2]], acts[op[4]], odt)
        elif op[0] == "up":
            t[op[2]] = orc.upsample2x(t[op[1]])
        elif op[0] == "relu":
            t[op[2]] = orc.add_act(t[op[1]], np.zeros_like(t[op[1]]), orc.ACT_RELU, odt)
    return {n: t[n] for n in outputs}
