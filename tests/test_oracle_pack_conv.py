"""Pins for the CPU oracle: mask / canonical pack (Section IV.C, "kernels with
similar patterns are grouped together"), storage rounding, the convolution
over pruned weights, and the layer grouping (Algorithm 1)."""
import numpy as np
import pytest
import torch
import torch.nn.functional as F

from oracle import rtoss_oracle as orc
from paper_2303_02191_b200 import synth


def _taps(m):
    return [t for t in range(9) if (m >> t) & 1]


# ---------------------------------------------------------------- rounding

def test_bf16_rounding_matches_torch():
    a = np.concatenate([synth.normal(9, 1, (20000,)), synth.normal(9, 2, (2000,), std=1e-30),
                        np.array([0.0, -0.0, 1.0, 65504.0, 3.3895314e38, 1e-45, np.inf, -np.inf], dtype=np.float32)])
    # exact half-way cases: 1 + 2^-8 (ties to even down), 1 + 3*2^-8 (ties to even up)
    a = np.concatenate([a, np.array([1 + 2.0 ** -8, 1 + 3 * 2.0 ** -8, -(1 + 2.0 ** -8)], dtype=np.float32)])
    want = torch.from_numpy(a).to(torch.bfloat16).to(torch.float32).numpy()
    got = orc.round_array(a, orc.DT_BF16)
    assert np.array_equal(got.view(np.uint32), want.view(np.uint32))


def test_f16_rounding_matches_numpy():
    a = np.concatenate([synth.normal(9, 3, (20000,)), synth.normal(9, 4, (5000,), std=1e-5),
                        synth.normal(9, 5, (5000,), std=1e-7), synth.normal(9, 6, (2000,), std=3e4),
                        np.array([0.0, -0.0, 65504.0, 65519.0, 65520.0, 1e-8, 2.0 ** -24, 2.0 ** -25, 3 * 2.0 ** -25,
                                  1 + 2.0 ** -11, 1 + 3 * 2.0 ** -11, np.inf, -np.inf], dtype=np.float32)])
    with np.errstate(over="ignore"):
        want = a.astype(np.float16).astype(np.float32)
    got = orc.round_array(a, orc.DT_F16)
    assert np.array_equal(got.view(np.uint32), want.view(np.uint32))
    assert orc.f32_to_f16_bits(1.0) == 0x3C00 and orc.f32_to_bf16_bits(1.0) == 0x3F80


# ---------------------------------------------------------------- mask / pack

@pytest.mark.parametrize("k,preset,dt", [(4, orc.PRESET_CENTRE8, orc.DT_F32), (3, orc.PRESET_CONN4, orc.DT_BF16),
                                          (2, orc.PRESET_CONN4, orc.DT_F16), (9, orc.PRESET_DENSE, orc.DT_BF16)])
def test_pack_3x3_invariants(k, preset, dt):
    masks = orc.pattern_preset(k, preset)
    P = len(masks)
    Cout, Cin = 37, 19
    w = synth.kaiming_weights(0, 5, Cout, Cin, 3)
    pid = orc.select_3x3(w, masks)
    wm = orc.mask_3x3(w, masks, pid)
    # exactly k kept positions per kernel, none removed entirely
    assert (np.count_nonzero(wm.reshape(-1, 9), axis=1) == k).all()
    kept = np.where(wm != 0, w, 0)
    assert np.array_equal(kept, wm)
    val, perm, off = orc.pack_3x3(w, masks, k, pid, dt)
    # values: ascending tap order, rounded by the library conversion
    tname = {orc.DT_F32: "f32", orc.DT_BF16: "bf16", orc.DT_F16: "f16"}[dt]
    for i in (0, 7, Cout * Cin - 1):
        co, ci = divmod(i, Cin)
        taps = _taps(int(masks[pid[co, ci]]))
        want = synth.round_like(w[co, ci].ravel()[taps], tname)
        assert np.array_equal(val[i * k:(i + 1) * k], want)
    # per input channel: stable sort of the filters by pattern id
    for ci in range(Cin):
        col = pid[:, ci]
        assert np.array_equal(perm[ci * Cout:(ci + 1) * Cout], np.argsort(col, kind="stable").astype(np.uint32))
        counts = np.bincount(col, minlength=P)
        assert np.array_equal(off[ci * (P + 1):(ci + 1) * (P + 1)], np.concatenate([[0], np.cumsum(counts)]))
    # round trip to dense == rounded masked weights, bit for bit
    wd = orc.unpack_3x3(val, Cout, Cin, masks, k, pid)
    assert np.array_equal(wd.view(np.uint32), synth.round_like(wm, tname).view(np.uint32))
    # compression = 9/k
    assert wm.size / np.count_nonzero(wd) == pytest.approx(9.0 / k, rel=1e-3)


@pytest.mark.parametrize("cout,cin", [(128, 256), (10, 7), (4, 2)])
def test_pack_1x1_round_trip(cout, cin):
    k = 3
    masks = orc.pattern_preset(k, orc.PRESET_CONN4)
    w = synth.kaiming_weights(0, 6, cout, cin, 1).reshape(cout, cin)
    pid1 = orc.select_1x1(w, masks)
    val1 = orc.pack_1x1(w, masks, k, pid1, orc.DT_BF16)
    G = (cout * cin) // 9
    assert len(val1) == G * k
    wd = orc.unpack_1x1(val1, cout, cin, masks, k, pid1)
    wm = synth.round_like(orc.mask_1x1(w, masks, pid1), "bf16")
    assert np.array_equal(wd.view(np.uint32), wm.view(np.uint32))
    assert np.count_nonzero(wd) == G * k


def test_stack_parameter_counts_and_compression():
    layers = synth.yolov5s_stack()
    assert len(layers) == 57
    assert sum(1 for l in layers if l["ksize"] == 3) == 18 and sum(1 for l in layers if l["stride"] == 2) == 7
    total = sum(l["cout"] * l["cin"] * l["ksize"] ** 2 for l in layers)
    kept = sum((l["cout"] * l["cin"] * 4) if l["ksize"] == 3 else ((l["cout"] * l["cin"]) // 9) * 4 for l in layers)
    assert abs(total - 6.985e6) < 5e3
    # Table 3 prints a 2.24x reduction for 4-entry patterns on YOLOv5s; the shape table gives 9/4
    assert total / kept == pytest.approx(2.25, abs=0.01)
    kept2 = sum((l["cout"] * l["cin"] * 2) if l["ksize"] == 3 else ((l["cout"] * l["cin"]) // 9) * 2 for l in layers)
    assert total / kept2 == pytest.approx(4.5, abs=0.01)   # paper: 4.4x for 2-entry patterns
    rn = synth.retinanet_r50fpn_stack()
    assert len(rn) == 100 and len({l["wid"] for l in rn}) == 68
    assert sum(1 for l in rn if l["ksize"] == 1) == 39
    assert (rn[-1]["H"], rn[-1]["W"]) == (7, 9)


# ---------------------------------------------------------------- convolution

def _torch_conv(x, wd, bias, stride, pad):
    y = F.conv2d(torch.from_numpy(x).double(), torch.from_numpy(wd).double(),
                 None if bias is None else torch.from_numpy(bias).double(), stride=stride, padding=pad)
    return y.numpy()


@pytest.mark.parametrize("stride", [1, 2])
@pytest.mark.parametrize("H,W", [(9, 7), (12, 16)])
def test_dense_table_is_ordinary_convolution(stride, H, W):
    masks = orc.pattern_preset(9, orc.PRESET_DENSE)
    x = synth.activations(1, 1, 2, 5, H, W)
    w = synth.kaiming_weights(1, 2, 6, 5, 3)
    b = synth.bias(1, 3, 6)
    pid = orc.select_3x3(w, masks)
    wd = orc.unpack_3x3(orc.pack_3x3(w, masks, 9, pid, orc.DT_F32)[0], 6, 5, masks, 9, pid)
    y = orc.conv3x3(x, wd, b, stride, orc.ACT_NONE, orc.DT_F32)
    ref = _torch_conv(x, w, b, stride, 1)
    assert y.shape == ref.shape
    assert np.abs(y - ref).max() < 1e-5


@pytest.mark.parametrize("stride", [1, 2])
def test_masked_conv_equals_library_conv_with_masked_weights(stride):
    masks = orc.pattern_preset(3, orc.PRESET_CONN4)
    x = synth.activations(2, 1, 1, 8, 11, 13)
    w = synth.kaiming_weights(2, 2, 4, 8, 3)
    pid = orc.select_3x3(w, masks)
    wm = orc.mask_3x3(w, masks, pid)
    y = orc.conv3x3(x, wm, None, stride, orc.ACT_NONE, orc.DT_F32)
    assert np.abs(y - _torch_conv(x, wm, None, stride, 1)).max() < 1e-5


def test_unit_impulse_reads_back_the_taps_without_flip():
    w = np.arange(1, 10, dtype=np.float32).reshape(1, 1, 3, 3)
    x = np.zeros((1, 1, 5, 5), dtype=np.float32)
    x[0, 0, 2, 2] = 1.0
    y = orc.conv3x3(x, w, None, 1, orc.ACT_NONE, orc.DT_F32)[0, 0]
    # cross-correlation: y[oy,ox] = w[2-oy+1, 2-ox+1] around the impulse
    assert np.array_equal(y[1:4, 1:4], w[0, 0][::-1, ::-1])
    assert not y[0].any() and not y[:, 0].any()
    # padding: impulse in the corner, stride 2 picks even input positions
    x[:] = 0
    x[0, 0, 0, 0] = 1.0
    y2 = orc.conv3x3(x, w, None, 2, orc.ACT_NONE, orc.DT_F32)[0, 0]
    assert y2.shape == (3, 3) and y2[0, 0] == w[0, 0, 1, 1] and not y2[1:].any() and not y2[:, 1:].any()


def test_packed_sparse_evaluation_equals_masked_dense():
    """Evaluate the convolution straight from (pid, val) in Python and compare
    with the oracle run on the unpacked dense weights."""
    k = 4
    masks = orc.pattern_preset(4, orc.PRESET_CENTRE8)
    N, Cin, Cout, H, W = 1, 3, 2, 6, 5
    x = synth.activations(3, 1, N, Cin, H, W)
    w = synth.kaiming_weights(3, 2, Cout, Cin, 3)
    b = synth.bias(3, 3, Cout)
    pid = orc.select_3x3(w, masks)
    val, _, _ = orc.pack_3x3(w, masks, k, pid, orc.DT_F32)
    wd = orc.unpack_3x3(val, Cout, Cin, masks, k, pid)
    y = orc.conv3x3(x, wd, b, 1, orc.ACT_NONE, orc.DT_F32)
    xp = np.pad(x.astype(np.float64), ((0, 0), (0, 0), (1, 1), (1, 1)))
    ref = np.zeros((N, Cout, H, W))
    for co in range(Cout):
        for ci in range(Cin):
            for j, t in enumerate(_taps(int(masks[pid[co, ci]]))):
                r, c = divmod(t, 3)
                ref[0, co] += float(val[(co * Cin + ci) * k + j]) * xp[0, ci, r:r + H, c:c + W]
        ref[0, co] += float(b[co])
    assert np.abs(y - ref).max() < 1e-6


def test_linearity_and_filter_permutation():
    masks = orc.pattern_preset(2, orc.PRESET_CONN4)
    x1, x2 = synth.activations(4, 1, 1, 4, 8, 8), synth.activations(4, 2, 1, 4, 8, 8)
    w = orc.mask_3x3(synth.kaiming_weights(4, 3, 5, 4, 3), masks, orc.select_3x3(synth.kaiming_weights(4, 3, 5, 4, 3), masks))
    f = lambda x, ww: orc.conv3x3(x, ww, None, 1, orc.ACT_NONE, orc.DT_F32)
    assert np.abs(f(x1 + x2, w) - (f(x1, w) + f(x2, w))).max() < 1e-5
    perm = np.array([3, 0, 4, 1, 2])
    assert np.array_equal(f(x1, w[perm]), f(x1, w)[:, perm])


def test_activations_bias_and_output_rounding():
    x = synth.activations(5, 1, 1, 3, 6, 6)
    w = synth.kaiming_weights(5, 2, 4, 3, 3)
    b = synth.bias(5, 3, 4)
    lin = _torch_conv(x, w, b, 1, 1)
    relu = orc.conv3x3(x, w, b, 1, orc.ACT_RELU, orc.DT_F32)
    silu = orc.conv3x3(x, w, b, 1, orc.ACT_SILU, orc.DT_F32)
    assert np.abs(relu - np.maximum(lin, 0)).max() < 1e-6
    assert np.abs(silu - lin / (1 + np.exp(-lin))).max() < 1e-6
    ybf = orc.conv3x3(x, w, b, 1, orc.ACT_SILU, orc.DT_BF16)
    want = torch.from_numpy(lin / (1 + np.exp(-lin))).to(torch.float32).to(torch.bfloat16).to(torch.float32).numpy()
    assert (ybf != want).mean() < 0.01      # double rounding may differ on rare half-way cases
    assert np.abs(ybf - want).max() <= np.abs(want).max() * 2.0 ** -8


@pytest.mark.parametrize("stride", [1, 2])
@pytest.mark.parametrize("cout,cin", [(6, 9), (5, 7)])
def test_1x1_conv_equals_library_conv_with_masked_matrix(stride, cout, cin):
    masks = orc.pattern_preset(3, orc.PRESET_CONN4)
    x = synth.activations(6, 1, 2, cin, 7, 9)
    w = synth.kaiming_weights(6, 2, cout, cin, 1).reshape(cout, cin)
    b = synth.bias(6, 3, cout)
    pid1 = orc.select_1x1(w, masks)
    wd = orc.unpack_1x1(orc.pack_1x1(w, masks, 3, pid1, orc.DT_F32), cout, cin, masks, 3, pid1)
    y = orc.conv1x1(x, wd, b, stride, orc.ACT_NONE, orc.DT_F32)
    ref = _torch_conv(x, wd.reshape(cout, cin, 1, 1), b, stride, 0)
    assert y.shape == ref.shape and np.abs(y - ref).max() < 1e-5
    # flat positions kept: k per full run, the tail zero
    flat = wd.ravel()
    G = (cout * cin) // 9
    assert all(np.count_nonzero(flat[9 * g:9 * g + 9]) == 3 for g in range(G)) and not flat[9 * G:].any()


def test_point_sampling_matches_full_tensor():
    x = synth.activations(7, 1, 2, 5, 9, 8)
    w = synth.kaiming_weights(7, 2, 4, 5, 3)
    b = synth.bias(7, 3, 4)
    y = orc.conv3x3(x, w, b, 2, orc.ACT_SILU, orc.DT_BF16)
    idx = np.array([[0, 0, 0, 0], [1, 3, 4, 3], [0, 2, 2, 1]], dtype=np.int32)
    pts = orc.conv_points(3, x, w, b, 2, orc.ACT_SILU, orc.DT_BF16, idx)
    assert np.array_equal(pts, y[idx[:, 0], idx[:, 1], idx[:, 2], idx[:, 3]])
    ref = _torch_conv(x, w, b, 2, 1)
    ref = ref / (1 + np.exp(-ref))
    assert np.abs(pts - ref[idx[:, 0], idx[:, 1], idx[:, 2], idx[:, 3]]).max() < 2e-2


# ---------------------------------------------------------------- layer grouping (Algorithm 1)

def _conv(cin, cout, ks, inputs):
    return dict(kind="conv", cin=cin, cout=cout, ksize=ks, inputs=inputs)


def test_grouping_hand_built_graphs():
    # chain of equal-shape 3x3 convs: one group, each the child of the previous one
    nodes = [_conv(8, 8, 3, []), _conv(8, 8, 3, [0]), _conv(8, 8, 3, [1])]
    parent, group, ng = orc.group_layers(nodes)
    assert parent.tolist() == [0, 0, 1] and group.tolist() == [0, 0, 0] and ng == 1
    # residual block: conv0 -> conv1 -> add(conv0, conv1) -> conv3; a 1x1 of another shape founds its own group
    nodes = [_conv(8, 8, 3, []), _conv(8, 8, 3, [0]), dict(kind="op", inputs=[0, 1]), _conv(8, 8, 3, [2]),
             _conv(8, 16, 1, [2]), _conv(8, 16, 1, [2])]
    parent, group, ng = orc.group_layers(nodes)
    assert parent.tolist() == [0, 0, -1, 0, 0, 0]          # DFS takes the first listed input first
    assert group.tolist() == [0, 0, -1, 0, 1, 2] and ng == 3
    # two independent roots
    nodes = [_conv(3, 4, 3, []), _conv(3, 4, 3, []), dict(kind="op", inputs=[1, 0]), _conv(3, 4, 3, [2])]
    parent, group, ng = orc.group_layers(nodes)
    assert parent.tolist() == [0, 1, -1, 1] and group.tolist() == [0, 1, -1, 1] and ng == 2


def test_grouping_invariants_on_the_yolov5s_graph():
    nodes = synth.yolov5s_graph()
    convs = [i for i, n in enumerate(nodes) if n["kind"] == "conv"]
    assert len(convs) == 57
    parent, group, ng = orc.group_layers(nodes)
    roots = [i for i in convs if parent[i] == i]
    assert roots == [convs[0]]                              # only the stem has no convolution upstream
    for i in convs:
        p = parent[i]
        assert nodes[p]["kind"] == "conv" and (p < i or p == i)
        a, b = nodes[i], nodes[p]
        same = (a["cin"], a["cout"], a["ksize"]) == (b["cin"], b["cout"], b["ksize"])
        assert (group[i] == group[p]) == same
    assert sorted(set(group[convs].tolist())) == list(range(ng))
    for g in range(ng):
        shapes = {(nodes[i]["cin"], nodes[i]["cout"], nodes[i]["ksize"]) for i in convs if group[i] == g}
        assert len(shapes) == 1
    assert all(group[i] == -1 and parent[i] == -1 for i in range(len(nodes)) if nodes[i]["kind"] != "conv")


# ---------------------------------------------------------------- glue operations (library routines as pins)

def test_glue_oracle_against_torch():
    x = synth.activations(60, 1, 2, 3, 9, 11)
    for k, s, p in ((5, 1, 2), (3, 2, 1), (2, 2, 0)):
        ref = F.max_pool2d(torch.from_numpy(x), k, s, p).numpy()
        assert np.array_equal(orc.maxpool2d(x, k, s, p), ref)
    assert np.array_equal(orc.upsample2x(x), np.repeat(np.repeat(x, 2, axis=2), 2, axis=3))
    y = synth.activations(60, 2, 2, 3, 9, 11)
    s_ = (x.astype(np.float64) + y.astype(np.float64))
    assert np.abs(orc.add_act(x, y, orc.ACT_NONE, orc.DT_F32) - s_).max() < 1e-6
    silu = orc.add_act(x, y, orc.ACT_SILU, orc.DT_BF16)
    want = torch.from_numpy((s_ / (1 + np.exp(-s_))).astype(np.float32)).to(torch.bfloat16).float().numpy()
    assert (silu != want).mean() < 0.01


def test_rel_err_on_hand_computed_cases():
    """The metric every convolution verdict rests on: max |y - ref| / max(|ref|, rms(ref)).
    ref = (6, -8, 0, 0): rms = sqrt((36 + 64) / 4) = 5 exactly.
      y = (6.3, -8.8, 1, 0): 0.3 / 6 = 0.05, 0.8 / 8 = 0.1, 1 / max(0, 5) = 0.2 (the element below the floor decides),
                             0 -> 0.2;
      y = (6, -10, 0.5, 0):  0, 2 / 8 = 0.25 (an element above the floor decides), 0.5 / 5 = 0.1 -> 0.25.
    A sum instead of the max in the denominator, the rms of y instead of ref's, a mean instead of the max over the
    elements, or no floor at all each miss at least one of the two."""
    ref = np.array([6.0, -8.0, 0.0, 0.0])
    assert abs(orc.rel_err(np.array([6.3, -8.8, 1.0, 0.0]), ref) - 0.2) < 1e-12
    assert abs(orc.rel_err(np.array([6.0, -10.0, 0.5, 0.0]), ref) - 0.25) < 1e-12
    assert orc.rel_err(ref, ref) == 0.0
    # shape does not matter, the floor is the rms of the whole reference tensor
    assert abs(orc.rel_err(np.array([[6.3, -8.8], [1.0, 0.0]]), ref.reshape(2, 2)) - 0.2) < 1e-12
    # the sampled-point form the large-layer tests spell out inline is the same formula
    got, r = np.array([6.3, -8.8, 1.0, 0.0]), ref
    rms = float(np.sqrt(np.mean(r ** 2)))
    assert abs(np.max(np.abs(got - r) / np.maximum(np.abs(r), max(rms, 1e-30))) - 0.2) < 1e-12
