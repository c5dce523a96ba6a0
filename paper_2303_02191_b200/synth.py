"""Seeded synthetic inputs and layer-shape tables.

This module holds no arithmetic of the pruning method: only random tensors of
the right shapes and value distributions (activations ~N(0,1), Kaiming-normal
weights, small biases) and tables of convolution shapes that stand in for the
paper's YOLOv5s and RetinaNet models (Section V.A of arXiv 2303.02191 names
the models and the 640x640 KITTI frames; the dataset and the trained weights
are not needed for the hot path, only the shapes).  Both the CUDA tests /
benchmark and the CPU oracle's tests draw their inputs from here.
"""
import math

import numpy as np


def _rng(seed, tensor_id):
    return np.random.default_rng([int(seed), int(tensor_id)])


def normal(seed, tensor_id, shape, std=1.0):
    """float32 N(0, std^2) tensor, a pure function of (seed, tensor_id, shape)."""
    a = _rng(seed, tensor_id).standard_normal(size=shape, dtype=np.float32)
    if std != 1.0:
        a *= np.float32(std)
    return a


def uniform_kernels(seed, n):
    """n random 3x3 kernels with entries uniform in [-1, 1) (the sample of the pattern usage ranking)."""
    return (_rng(seed, 424242).random(size=(n, 9), dtype=np.float32) * np.float32(2.0) - np.float32(1.0)).astype(np.float32)


def activations(seed, tensor_id, N, C, H, W):
    """NCHW float32 activations ~N(0,1)."""
    return normal(seed, 2 * tensor_id, (N, C, H, W))


def kaiming_weights(seed, tensor_id, cout, cin, ksize):
    """[Cout,Cin,ks,ks] float32, std = sqrt(2 / (Cin*ks*ks))."""
    return normal(seed, 2 * tensor_id + 1, (cout, cin, ksize, ksize), std=math.sqrt(2.0 / (cin * ksize * ksize)))


def bias(seed, tensor_id, cout):
    return normal(seed + 7919, tensor_id, (cout,), std=0.1)


def round_like(a, dtype_name):
    """Round a float32 array once to 'f32' | 'bf16' | 'f16' storage and return
    it as float32 (library conversion: torch on CPU)."""
    if dtype_name == "f32":
        return np.ascontiguousarray(a, dtype=np.float32)
    import torch
    td = {"bf16": torch.bfloat16, "f16": torch.float16}[dtype_name]
    return torch.from_numpy(np.ascontiguousarray(a, dtype=np.float32)).to(td).to(torch.float32).numpy()


# --------------------------------------------------------------------------
# Layer tables.  Each entry: dict(name, ksize, stride, cin, cout, H, W, act,
# wid) with H, W the INPUT size and wid the weight-tensor id (calls sharing a
# wid share one weight tensor).
# --------------------------------------------------------------------------

def _L(name, ksize, stride, cin, cout, H, W, act, wid):
    return dict(name=name, ksize=ksize, stride=stride, cin=cin, cout=cout, H=H, W=W, act=act, wid=wid)


def out_hw(H, W, stride):
    return (H - 1) // stride + 1, (W - 1) // stride + 1


def yolov5s_stack(H0=640, W0=640):
    """YOLOv5s-shaped backbone + neck: 57 convolutions (18 3x3, 39 1x1), SiLU
    after each, widths 32..512, detection head excluded."""
    layers = []

    def add(name, ks, s, cin, cout, H, W):
        layers.append(_L(name, ks, s, cin, cout, H, W, "silu", len(layers)))
        return out_hw(H, W, s)

    def c3(tag, c1, c2, n, H, W):
        h = c2 // 2
        add(tag + ".cv1", 1, 1, c1, h, H, W)
        add(tag + ".cv2", 1, 1, c1, h, H, W)
        for i in range(n):
            add("%s.m%d.cv1" % (tag, i), 1, 1, h, h, H, W)
            add("%s.m%d.cv2" % (tag, i), 3, 1, h, h, H, W)
        add(tag + ".cv3", 1, 1, c2, c2, H, W)

    H, W = add("stem", 3, 2, 3, 32, H0, W0)
    H, W = add("down1", 3, 2, 32, 64, H, W)
    c3("c3_1", 64, 64, 1, H, W)
    H, W = add("down2", 3, 2, 64, 128, H, W)
    H8, W8 = H, W
    c3("c3_2", 128, 128, 2, H, W)
    H, W = add("down3", 3, 2, 128, 256, H, W)
    H16, W16 = H, W
    c3("c3_3", 256, 256, 3, H, W)
    H, W = add("down4", 3, 2, 256, 512, H, W)
    H32, W32 = H, W
    c3("c3_4", 512, 512, 1, H, W)
    add("sppf.cv1", 1, 1, 512, 256, H, W)
    add("sppf.cv2", 1, 1, 1024, 512, H, W)
    add("neck.cv1", 1, 1, 512, 256, H32, W32)
    c3("neck.c3_1", 512, 256, 1, H16, W16)
    add("neck.cv2", 1, 1, 256, 128, H16, W16)
    c3("neck.c3_2", 256, 128, 1, H8, W8)
    add("neck.down1", 3, 2, 128, 128, H8, W8)
    c3("neck.c3_3", 256, 256, 1, H16, W16)
    add("neck.down2", 3, 2, 256, 256, H16, W16)
    c3("neck.c3_4", 512, 512, 1, H32, W32)
    return layers


def retinanet_r50fpn_stack(H0=800, W0=1088):
    """RetinaNet ResNet-50-FPN-shaped conv stack after the 7x7 stem and the
    3x3/s2 max-pool (so it starts at 64 x H0/4 x W0/4): bottlenecks [3,4,6,3],
    FPN P3..P7 at 256 channels, two towers of 4 x (3x3 256->256 + ReLU) applied
    to the five levels with shared weights.  100 calls on 68 weight tensors."""
    layers = []
    nw = [0]

    def add(name, ks, s, cin, cout, H, W, act, wid=None):
        if wid is None:
            wid = nw[0]
            nw[0] += 1
        layers.append(_L(name, ks, s, cin, cout, H, W, act, wid))
        return out_hw(H, W, s)

    H, W = H0 // 4, W0 // 4
    cin = 64
    feats = {}
    for si, (nblk, w) in enumerate(zip([3, 4, 6, 3], [64, 128, 256, 512])):
        for b in range(nblk):
            s = 2 if (b == 0 and si > 0) else 1
            tag = "layer%d.%d" % (si + 1, b)
            add(tag + ".conv1", 1, 1, cin, w, H, W, "relu")
            Ho, Wo = add(tag + ".conv2", 3, s, w, w, H, W, "relu")
            add(tag + ".conv3", 1, 1, w, 4 * w, Ho, Wo, "relu")
            if b == 0:
                add(tag + ".downsample", 1, s, cin, 4 * w, H, W, "none")
            cin = 4 * w
            H, W = Ho, Wo
        feats[si] = (cin, H, W)
    levels = []
    for si in (1, 2, 3):
        c, h, w_ = feats[si]
        add("fpn.lateral%d" % (si + 2), 1, 1, c, 256, h, w_, "none")
    for si in (1, 2, 3):
        c, h, w_ = feats[si]
        add("fpn.output%d" % (si + 2), 3, 1, 256, 256, h, w_, "none")
        levels.append((h, w_))
    h, w_ = levels[-1]
    h6, w6 = add("fpn.p6", 3, 2, 256, 256, h, w_, "none")
    levels.append((h6, w6))
    h7, w7 = add("fpn.p7", 3, 2, 256, 256, h6, w6, "none")
    levels.append((h7, w7))
    for tower in ("cls", "box"):
        wids = []
        for i in range(4):
            wids.append(nw[0])
            nw[0] += 1
        for li, (h, w_) in enumerate(levels):
            for i in range(4):
                add("%s_tower%d.p%d" % (tower, i, li + 3), 3, 1, 256, 256, h, w_, "relu", wid=wids[i])
    return layers


def independent_sets(layers):
    """Launch units of a layer table: lists of layer indices, in execution order, whose members do not depend on one
    another in the network the table was taken from, so that they may run side by side (one grouped launch).
      YOLOv5s-shaped: the two 1x1 branches (cv1, cv2) that open a C3 block read the same input.
      RetinaNet-shaped: tower layer i of both towers on all five pyramid levels (each needs only tower layer i-1 of
      its own tower and level); the three 3x3 pyramid outputs; the three 1x1 laterals; the first 1x1 of a stage's first
      bottleneck and that block's 1x1 projection (both read the block input).
    Every other layer is a unit of its own."""
    import re
    key_of = {}
    for i, L in enumerate(layers):
        n = L["name"]
        m = re.match(r"(cls|box)_tower(\d)\.p\d$", n)
        if m:
            key_of[i] = "tower%s" % m.group(2)
        elif re.match(r"fpn\.output\d$", n):
            key_of[i] = "fpn.output"
        elif re.match(r"fpn\.lateral\d$", n):
            key_of[i] = "fpn.lateral"
        elif re.match(r"layer\d\.0\.(conv1|downsample)$", n):
            key_of[i] = n.rsplit(".", 1)[0] + ".in"
        elif re.match(r".*c3_\d\.cv[12]$", n):
            key_of[i] = n.rsplit(".", 1)[0] + ".in"
    units, at = [], {}
    for i in range(len(layers)):
        k = key_of.get(i)
        if k is None:
            units.append([i])
        elif k in at:
            units[at[k]].append(i)
        else:
            at[k] = len(units)
            units.append([i])
    return units


def chained_units(layers):
    """independent_sets with successive tower layers merged: -> (units, afters).  In the RetinaNet-shaped network
    tower layer i of a level reads tower layer i - 1 of the same tower and level and nothing else, so layers 0 + 1 and
    2 + 3 of both towers on all levels (twenty convolutions each) can share a launch whose members wait for one another
    (rtoss_conv_chain).  afters[u] is None for a unit of independent convolutions, else one bit mask per member: bit j
    set when the member has to wait for member j of the same unit."""
    import re
    units = independent_sets(layers)
    key = []
    for u in units:
        m = re.match(r"(cls|box)_tower(\d)\.p\d$", layers[u[0]]["name"])
        key.append(int(m.group(2)) if m else None)
    out_units, afters, skip = [], [], set()
    for ui, u in enumerate(units):
        if ui in skip:
            continue
        nxt = None
        if key[ui] is not None and key[ui] % 2 == 0:
            for vi in range(ui + 1, len(units)):
                if key[vi] == key[ui] + 1:
                    nxt = vi
                    break
        if nxt is None:
            out_units.append(list(u))
            afters.append(None)
            continue
        skip.add(nxt)
        merged = list(u) + list(units[nxt])
        name_at = {layers[i]["name"]: q for q, i in enumerate(merged)}
        after = []
        for i in merged:
            m = re.match(r"(cls|box)_tower(\d)(\.p\d)$", layers[i]["name"])
            prev = "%s_tower%d%s" % (m.group(1), int(m.group(2)) - 1, m.group(3))
            after.append(1 << name_at[prev] if prev in name_at else 0)
        out_units.append(merged)
        afters.append(after)
    return out_units, afters


def layer_nnz_flops(layer, N, k):
    """2 * (kept multiply-adds) of one call at batch N with k kept taps."""
    Ho, Wo = out_hw(layer["H"], layer["W"], layer["stride"])
    if layer["ksize"] == 3:
        kept = layer["cout"] * layer["cin"] * k
    else:
        kept = ((layer["cout"] * layer["cin"]) // 9) * k
    return 2.0 * kept * N * Ho * Wo


def layer_bytes(layer, N, k, elem):
    """Algorithmic bytes of one call: x once, y once, packed values + pattern
    ids, bias."""
    Ho, Wo = out_hw(layer["H"], layer["W"], layer["stride"])
    nk = layer["cout"] * layer["cin"] if layer["ksize"] == 3 else (layer["cout"] * layer["cin"]) // 9
    return (N * layer["cin"] * layer["H"] * layer["W"] * elem + N * layer["cout"] * Ho * Wo * elem
            + nk * (k * elem + 1) + 4 * layer["cout"])


def yolov5s_graph():
    """The YOLOv5s-shaped stack as a DAG for the layer-grouping step: a list of
    nodes dict(kind='conv'|'op', cout, cin, ksize, inputs=[node ids]) in
    topological order.  'op' nodes are the glue (add, concat, pool, upsample)."""
    nodes = []

    def conv(cin, cout, ks, inputs):
        nodes.append(dict(kind="conv", cin=cin, cout=cout, ksize=ks, inputs=list(inputs)))
        return len(nodes) - 1

    def op(inputs):
        nodes.append(dict(kind="op", inputs=list(inputs)))
        return len(nodes) - 1

    def c3(x, c1, c2, n, shortcut):
        h = c2 // 2
        a = conv(c1, h, 1, [x])
        b = conv(c1, h, 1, [x])
        y = a
        for _ in range(n):
            m1 = conv(h, h, 1, [y])
            m2 = conv(h, h, 3, [m1])
            y = op([y, m2]) if shortcut else m2
        cat = op([y, b])
        return conv(c2, c2, 1, [cat])

    x = conv(3, 32, 3, [])
    x = conv(32, 64, 3, [x])
    x = c3(x, 64, 64, 1, True)
    x = conv(64, 128, 3, [x])
    p3 = c3(x, 128, 128, 2, True)
    x = conv(128, 256, 3, [p3])
    p4 = c3(x, 256, 256, 3, True)
    x = conv(256, 512, 3, [p4])
    x = c3(x, 512, 512, 1, True)
    s1 = conv(512, 256, 1, [x])
    m1 = op([s1]); m2 = op([m1]); m3 = op([m2])
    cat = op([s1, m1, m2, m3])
    p5 = conv(1024, 512, 1, [cat])
    n1 = conv(512, 256, 1, [p5])
    up = op([n1])
    cat = op([up, p4])
    x = c3(cat, 512, 256, 1, False)
    n2 = conv(256, 128, 1, [x])
    up = op([n2])
    cat = op([up, p3])
    o3 = c3(cat, 256, 128, 1, False)
    d = conv(128, 128, 3, [o3])
    cat = op([d, n2])
    o4 = c3(cat, 256, 256, 1, False)
    d = conv(256, 256, 3, [o4])
    cat = op([d, n1])
    c3(cat, 512, 512, 1, False)
    return nodes
