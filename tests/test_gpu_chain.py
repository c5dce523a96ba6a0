"""GPU parity of rtoss_conv_chain: convolutions that depend on one another in ONE launch (the CTAs wait inside the kernel
for the tiles of the layers a layer reads).  Every layer's output is compared with the CPU oracle applied to the input
that layer actually read on the GPU, so a tile fetched before its producer had written it fails the layer's own bound;
the intermediate buffers are filled with NaN before every run to make such a read loud."""
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


def _table(k):
    return orc.pattern_preset(k, orc.PRESET_CENTRE8 if k == 4 else orc.PRESET_CONN4)


class Net:
    """A small program of convolutions over named NHWC buffers.  spec: (name, ks, Cout, stride, act, src, residual or None)."""

    def __init__(self, seed, N, C0, H, W, spec, dt="bf16", k=4, path=0):
        self.c, self.N, self.dt, self.k, self.spec, self.path = gu.ctx(), N, dt, k, spec, path
        self.masks = _table(k)
        self.shape = {"in": (C0, H, W)}
        self.layers = {}
        for tid, (name, ks, Cout, stride, act, src, res) in enumerate(spec):
            Cin, Hi, Wi = self.shape[src]
            Ho, Wo = synth.out_hw(Hi, Wi, stride)
            self.shape[name] = (Cout, Ho, Wo)
            w = synth.kaiming_weights(seed, tid, Cout, Cin, ks)
            b = synth.bias(seed, tid, Cout)
            wd = gu.to_dev(w, "f32")
            pid = self.c.rtoss_select_patterns(wd, ks, self.masks, k)
            packed = self.c.rtoss_pack(wd, ks, self.masks, k, pid, rt.DTYPE_NAMES[dt])
            _, wdense, _ = gu.oracle_weights(w, ks, self.masks, k, dt)
            self.layers[name] = dict(packed=packed, bias=torch.from_numpy(b).cuda(), b=b, wdense=wdense)
        self.x0 = synth.round_like(synth.activations(seed, 99, N, C0, H, W), dt)
        self.t = {n: torch.zeros((N, h, w, c), dtype=gu.TORCH_DT[dt], device="cuda") for n, (c, h, w) in self.shape.items()}
        self.t["in"].copy_(gu.to_dev(self.x0, dt, "nhwc"))

    def poison(self):
        for n, t in self.t.items():
            if n != "in":
                t.fill_(float("nan"))

    def items(self):
        out = []
        for (name, ks, Cout, stride, act, src, res) in self.spec:
            L = self.layers[name]
            _, Hi, Wi = self.shape[src]
            out.append(self.c.conv_item(L["packed"], self.t[src], self.t[name], self.N, Hi, Wi, stride, rt.NHWC, ACT[act], L["bias"],
                                        residual=self.t[res] if res else None, path=self.path))
        return out

    def read(self):
        return {n: gu.from_dev(t, "nhwc") for n, t in self.t.items()}

    def check_each_layer(self, got):
        """Every layer against the oracle on the inputs the GPU run had."""
        a = {"none": orc.ACT_NONE, "relu": orc.ACT_RELU, "silu": orc.ACT_SILU}
        for (name, ks, Cout, stride, act, src, res) in self.spec:
            L = self.layers[name]
            assert np.isfinite(got[name]).all(), name
            if res:
                ref = gu.oracle_conv(ks, got[src], L["wdense"], L["b"], stride, "none", self.dt)
                ref = orc.add_act(ref, got[res], a[act], gu.ORC_DT[self.dt])
            else:
                ref = gu.oracle_conv(ks, got[src], L["wdense"], L["b"], stride, act, self.dt)
            err = orc.rel_err(got[name], ref)
            assert err <= gu.TOL[self.dt], (name, err)

    def close(self):
        for L in self.layers.values():
            L["packed"].close()


# two bottleneck blocks, the first with a stride-2 3x3 and a stride-2 projection (the shape of a ResNet stage's entry)
STAGE = [
    ("a1", 1, 128, 1, "relu", "in", None),
    ("ad", 1, 256, 2, "none", "in", None),
    ("a2", 3, 128, 2, "relu", "a1", None),
    ("a3", 1, 256, 1, "relu", "a2", "ad"),
    ("b1", 1, 128, 1, "relu", "a3", None),
    ("b2", 3, 128, 1, "relu", "b1", None),
    ("b3", 1, 256, 1, "relu", "b2", "a3"),
]


def test_a_stage_of_bottleneck_blocks_is_one_launch():
    # (RTOSS_PATH_TENSOR keeps the small 3x3 layers in the shared launch; left to itself the library would give each a
    # launch of its own, cut along the channels: the second run below)
    net = Net(81, 2, 96, 40, 56, STAGE, path=rt.PATH_TENSOR)
    c = net.c
    items = net.items()
    after = rt.rtoss_chain_deps(items)
    assert after == [0, 0, 0b1, 0b110, 0b1000, 0b10000, 0b101000]
    net.poison()
    assert c.rtoss_conv_chain(items) == 1
    torch.cuda.synchronize()
    assert c.rtoss_device_status() == 0
    got = net.read()
    net.check_each_layer(got)
    # the same bits every time, also with the dependencies spelled out and through a replayed graph
    for how in ("again", "explicit", "graph"):
        net.poison()
        if how == "graph":
            g = torch.cuda.CUDAGraph()
            side = torch.cuda.Stream()
            side.wait_stream(torch.cuda.current_stream())
            with torch.cuda.stream(side):
                c.rtoss_conv_chain(items)
            torch.cuda.current_stream().wait_stream(side)
            torch.cuda.synchronize()
            net.poison()
            with torch.cuda.graph(g):
                c.rtoss_conv_chain(items)
            for _ in range(3):
                g.replay()
        else:
            assert c.rtoss_conv_chain(items, after if how == "explicit" else None) == 1
        torch.cuda.synchronize()
        again = net.read()
        for name in net.shape:
            assert np.array_equal(again[name].view(np.uint32), got[name].view(np.uint32)), (how, name)
    # left to choose, the library takes the small 3x3 layers out of the shared launches
    auto = Net(81, 2, 96, 40, 56, STAGE)
    auto.poison()
    assert 1 < c.rtoss_conv_chain(auto.items()) < len(STAGE)
    torch.cuda.synchronize()
    auto.check_each_layer(auto.read())
    auto.close()
    # one call per convolution, in order: the same network (other tile plans, so other summation order)
    net.poison()
    for it in items:
        assert c.rtoss_conv_group([it]) == 1
    torch.cuda.synchronize()
    single = net.read()
    net.check_each_layer(single)
    assert orc.rel_err(single["b3"], got["b3"]) <= 0.05
    assert c.rtoss_device_status() == 0
    net.close()


def test_tower_layers_follow_their_own_level_only():
    """Two tower layers over three pyramid levels with shared weights: layer 1 of a level waits for layer 0 of that level,
    not for the other levels, and everything is one launch."""
    c = gu.ctx()
    masks, k, dt = _table(4), 4, "bf16"
    packs = []
    for tid in range(2):
        w = synth.kaiming_weights(82, tid, 256, 256, 3)
        wd = gu.to_dev(w, "f32")
        packed = c.rtoss_pack(wd, 3, masks, k, c.rtoss_select_patterns(wd, 3, masks, k), rt.DTYPE_NAMES[dt])
        packs.append(dict(packed=packed, wdense=gu.oracle_weights(w, 3, masks, k, dt)[1], b=synth.bias(82, tid, 256)))
    levels = [(40, 52), (20, 26), (5, 7)]
    N = 2
    xs = [synth.round_like(synth.activations(82, 10 + i, N, 256, h, w), dt) for i, (h, w) in enumerate(levels)]
    t_in = [gu.to_dev(x, dt, "nhwc") for x in xs]
    t_mid = [torch.full((N, h, w, 256), float("nan"), dtype=torch.bfloat16, device="cuda") for (h, w) in levels]
    t_out = [torch.full((N, h, w, 256), float("nan"), dtype=torch.bfloat16, device="cuda") for (h, w) in levels]
    bias = [torch.from_numpy(p["b"]).cuda() for p in packs]
    items = []
    for i, (h, w) in enumerate(levels):
        items.append(c.conv_item(packs[0]["packed"], t_in[i], t_mid[i], N, h, w, 1, rt.NHWC, ACT["relu"], bias[0], path=rt.PATH_TENSOR))
    for i, (h, w) in enumerate(levels):
        items.append(c.conv_item(packs[1]["packed"], t_mid[i], t_out[i], N, h, w, 1, rt.NHWC, ACT["relu"], bias[1], path=rt.PATH_TENSOR))
    assert rt.rtoss_chain_deps(items) == [0, 0, 0, 0b001, 0b010, 0b100]
    assert c.rtoss_conv_chain(items) == 1
    torch.cuda.synchronize()
    assert c.rtoss_device_status() == 0
    for i in range(3):
        mid = gu.from_dev(t_mid[i], "nhwc")
        out = gu.from_dev(t_out[i], "nhwc")
        assert orc.rel_err(mid, gu.oracle_conv(3, xs[i], packs[0]["wdense"], packs[0]["b"], 1, "relu", dt)) <= gu.TOL[dt]
        assert orc.rel_err(out, gu.oracle_conv(3, mid, packs[1]["wdense"], packs[1]["b"], 1, "relu", dt)) <= gu.TOL[dt]
    for p in packs:
        p["packed"].close()


def test_fp32_chain_and_buffer_reuse():
    """fp32 (three tf32 products per tap) through a chain whose third layer writes over the first layer's input: the
    writer waits for the reader."""
    spec = [
        ("p", 3, 96, 1, "silu", "in", None),
        ("q", 1, 96, 1, "none", "p", None),
    ]
    net = Net(83, 1, 96, 18, 22, spec, dt="f32", path=rt.PATH_TENSOR)
    c = net.c
    Lr = net.layers["q"]
    items = net.items()
    # a third convolution q -> "in" (same shape as the input): it must wait for p, which reads "in", and for q
    w = synth.kaiming_weights(83, 7, 96, 96, 3)
    wd = gu.to_dev(w, "f32")
    packed = c.rtoss_pack(wd, 3, net.masks, net.k, c.rtoss_select_patterns(wd, 3, net.masks, net.k), rt.DTYPE_NAMES["f32"])
    wdense = gu.oracle_weights(w, 3, net.masks, net.k, "f32")[1]
    b = synth.bias(83, 7, 96)
    items.append(c.conv_item(packed, net.t["q"], net.t["in"], 1, 18, 22, 1, rt.NHWC, ACT["relu"], torch.from_numpy(b).cuda(),
                             path=rt.PATH_TENSOR))
    assert rt.rtoss_chain_deps(items) == [0, 0b01, 0b11]
    net.poison()
    assert c.rtoss_conv_chain(items) == 1
    torch.cuda.synchronize()
    assert c.rtoss_device_status() == 0
    got = net.read()
    ref_p = gu.oracle_conv(3, net.x0, net.layers["p"]["wdense"], net.layers["p"]["b"], 1, "silu", "f32")
    assert orc.rel_err(got["p"], ref_p) <= gu.TOL["f32"]
    assert orc.rel_err(got["q"], gu.oracle_conv(1, got["p"], Lr["wdense"], Lr["b"], 1, "none", "f32")) <= gu.TOL["f32"]
    assert orc.rel_err(got["in"], gu.oracle_conv(3, got["q"], wdense, b, 1, "relu", "f32")) <= gu.TOL["f32"]
    packed.close()
    net.close()


def test_items_the_shared_launch_does_not_take_run_in_order():
    """A narrow 1x1 layer (positions on M) in front: it goes out on its own, the rest as one launch, same results."""
    spec = [
        ("u", 1, 48, 1, "relu", "in", None),      # 48 filters: not a member of shared launches
        ("v", 3, 128, 1, "relu", "u", None),
        ("w", 1, 128, 1, "none", "v", None),
    ]
    net = Net(84, 2, 64, 20, 20, spec)
    net.poison()
    assert net.c.rtoss_conv_chain(net.items()) == 2      # u on its own, then v and w together
    torch.cuda.synchronize()
    net.check_each_layer(net.read())
    with pytest.raises(rt.RtossError):
        net.c.rtoss_conv_chain(net.items(), [0, 0b10, 0])   # an item ordered behind itself / a later one
    assert net.c.rtoss_device_status() == 0
    net.close()
