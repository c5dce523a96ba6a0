"""GPU parity: the CUDA path, called through the C ABI, against the CPU oracle
on the same seeded inputs.  Pattern ids and packed arrays must match bit for
bit; convolution outputs within 1e-4 (fp32) / 2e-2 (bf16, fp16 inputs with fp32
accumulation), relative error floored by the tensor's RMS."""
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
    if k == 4:
        return orc.pattern_preset(4, orc.PRESET_CENTRE8)
    if k == 9:
        return orc.pattern_preset(9, orc.PRESET_DENSE)
    return orc.pattern_preset(k, orc.PRESET_CONN4)


# ---- the small single-layer configuration: 3x3, 32->32, 32x32, fp32, 8 centre patterns
@pytest.mark.parametrize("layout", ["nchw", "nhwc"])
@pytest.mark.parametrize("act", ["none", "silu"])
def test_config1_fp32(layout, act):
    gu.check_layer(0, 1, 3, 1, 32, 32, 32, 32, 1, 4, _table(4), "f32", act, layout)


# ---- the 128-channel 80x80 bf16 layer, 3- and 2-entry patterns, one image in full
@pytest.mark.parametrize("k", [3, 2, 4])
def test_config2_3x3_bf16_one_image(k):
    gu.check_layer(0, 2, 3, 1, 128, 128, 80, 80, 1, k, _table(k), "bf16", "silu")


@pytest.mark.parametrize("k", [3, 2, 4])
def test_config2_1x1_bf16_one_image(k):
    gu.check_layer(0, 3, 1, 1, 256, 128, 80, 80, 1, k, _table(k), "bf16", "silu")


def _sampled_parity(ksize, N, Cin, Cout, H, W, stride, k, dt, act, npts=4000, layout="nchw"):
    masks = _table(k)
    x = synth.round_like(synth.activations(0, 40 + ksize, N, Cin, H, W), dt)
    w = synth.kaiming_weights(0, 40 + ksize, Cout, Cin, ksize)
    b = synth.bias(0, 40 + ksize, Cout)
    pid_g, packed = gu.select_pack(w, ksize, masks, k, dt)
    pid_o, wd, _ = gu.oracle_weights(w, ksize, masks, k, dt)
    assert np.array_equal(pid_g, pid_o.ravel())
    y = gu.run_conv(packed, ksize, x, dt, stride, act, b, layout)
    Ho, Wo = synth.out_hw(H, W, stride)
    rng = np.random.default_rng(5)
    idx = np.stack([rng.integers(0, N, npts), rng.integers(0, Cout, npts), rng.integers(0, Ho, npts),
                    rng.integers(0, Wo, npts)], axis=1).astype(np.int32)
    # always include the four corners and the last pixel of the last image/filter
    idx[:5] = [[0, 0, 0, 0], [0, 0, 0, Wo - 1], [0, 0, Ho - 1, 0], [N - 1, Cout - 1, Ho - 1, Wo - 1], [N - 1, 0, Ho - 1, Wo - 1]]
    a = {"none": orc.ACT_NONE, "relu": orc.ACT_RELU, "silu": orc.ACT_SILU}[act]
    ref = orc.conv_points(ksize, x, wd, b, stride, a, gu.ORC_DT[dt], idx)
    got = y[idx[:, 0], idx[:, 1], idx[:, 2], idx[:, 3]]
    rms = float(np.sqrt(np.mean(ref.astype(np.float64) ** 2)))
    err = np.max(np.abs(got - ref) / np.maximum(np.abs(ref), rms))
    assert err <= gu.TOL[dt], err
    assert np.isfinite(y).all()
    packed.close()


@pytest.mark.parametrize("k", [3, 2])
def test_config2_3x3_full_batch_sampled(k):
    _sampled_parity(3, 8, 128, 128, 80, 80, 1, k, "bf16", "silu")


def test_config2_1x1_full_batch_sampled():
    _sampled_parity(1, 8, 256, 128, 80, 80, 1, 3, "bf16", "silu")


# ---- shapes with ragged tiles, strides, odd channel counts, other dtypes / layouts / epilogues
SHAPES_3x3 = [
    # N, Cin, Cout, H, W, stride, k, dt, act, layout, bias
    (2, 3, 32, 33, 41, 2, 4, "bf16", "silu", "nchw", True),     # stem-like: Cin=3, stride 2, odd size
    (1, 13, 20, 7, 9, 1, 3, "f32", "relu", "nchw", True),       # channels not multiples of the tiles
    (1, 16, 40, 13, 17, 2, 2, "f16", "none", "nhwc", False),
    (2, 24, 33, 25, 34, 1, 4, "bf16", "relu", "nhwc", True),
    (1, 8, 8, 1, 1, 1, 4, "f32", "none", "nchw", True),         # single pixel
    (1, 1, 1, 5, 5, 1, 9, "f32", "none", "nchw", False),        # single kernel, dense table
    (1, 32, 64, 40, 40, 2, 4, "bf16", "silu", "nchw", True),
    (3, 16, 16, 20, 20, 1, 9, "bf16", "silu", "nchw", True),    # k = 9: no pruning
    (1, 9, 5, 12, 100, 1, 5, "f32", "silu", "nchw", True),      # 5-entry patterns, wide image
    (1, 64, 64, 16, 16, 2, 1, "f16", "relu", "nchw", True),     # 1-entry patterns
    (2, 16, 32, 25, 34, 1, 4, "bf16", "relu", "nchw", True),    # rows 68 bytes: 4-byte async copies
    (1, 24, 32, 50, 68, 2, 4, "bf16", "relu", "nchw", True),    # rows 136 bytes: 8-byte async copies
    (1, 8, 16, 11, 6, 1, 3, "f32", "none", "nchw", True),       # fp32 rows of 24 bytes
    (1, 16, 24, 30, 22, 1, 4, "f32", "silu", "nhwc", True),     # fp32 NHWC, two 16-byte vectors per pixel
    (1, 40, 36, 200, 272, 2, 4, "bf16", "relu", "nchw", False), # large image, stride 2, many tiles
    (2, 3, 40, 20, 22, 1, 3, "f16", "silu", "nhwc", True),      # 3-channel stem kernel, NHWC, ragged filter block
    (1, 4, 64, 16, 16, 2, 2, "bf16", "relu", "nhwc", False),    # 4-channel stem kernel, vector stores
    (1, 2, 32, 9, 9, 1, 4, "f32", "none", "nchw", True),
    (2, 3, 32, 32, 48, 2, 4, "bf16", "silu", "nhwc", True),     # detector stem: 16-byte window loads, staged stores, 2 blocks
    (1, 3, 32, 24, 40, 2, 4, "f16", "relu", "nhwc", True),      # the same in fp16
    (1, 3, 64, 16, 16, 2, 4, "bf16", "silu", "nhwc", True),     # two filter blocks: staged stores into 128-byte pixels
    (1, 3, 32, 18, 20, 2, 4, "bf16", "silu", "nhwc", True),     # rows of 20 pixels: element loads, 10 outputs a row: direct stores
    (1, 3, 32, 12, 16, 1, 4, "bf16", "none", "nhwc", True),     # stride 1: element loads, staged stores
    (8, 3, 32, 480, 480, 2, 4, "bf16", "silu", "nhwc", True),   # more groups than one round of the grid
]


@pytest.mark.parametrize("case", SHAPES_3x3, ids=lambda c: "-".join(str(v) for v in c))
def test_conv3x3_shapes(case):
    N, Cin, Cout, H, W, s, k, dt, act, layout, ub = case
    masks = _table(k) if k in (2, 3, 4, 9) else orc.pattern_preset(k, orc.PRESET_CONN4)
    gu.check_layer(1, 100 + Cin, 3, N, Cin, Cout, H, W, s, k, masks, dt, act, layout, ub)


SHAPES_1x1 = [
    (2, 64, 32, 20, 20, 1, 4, "bf16", "silu", "nchw", True),
    (1, 256, 512, 25, 34, 2, 4, "bf16", "none", "nchw", True),  # stride-2 downsample branch
    (1, 7, 5, 9, 11, 1, 3, "f32", "relu", "nchw", True),        # 35 weights: 3 runs + 8 left over
    (1, 2, 4, 6, 6, 1, 2, "f32", "none", "nchw", True),         # fewer than 9 weights: everything pruned
    (2, 40, 24, 13, 17, 1, 2, "f16", "relu", "nhwc", False),
    (1, 128, 64, 33, 33, 2, 3, "bf16", "silu", "nhwc", True),
    (1, 72, 16, 40, 40, 1, 9, "f32", "none", "nchw", True),     # dense table: plain 1x1 conv minus the tail rule
]


@pytest.mark.parametrize("case", SHAPES_1x1, ids=lambda c: "-".join(str(v) for v in c))
def test_conv1x1_shapes(case):
    N, Cin, Cout, H, W, s, k, dt, act, layout, ub = case
    gu.check_layer(2, 200 + Cin, 1, N, Cin, Cout, H, W, s, k, _table(k), dt, act, layout, ub)


def test_channel_slice_output_and_untouched_neighbours():
    masks = _table(4)
    x = synth.round_like(synth.activations(3, 1, 1, 16, 12, 12), "bf16")
    w = synth.kaiming_weights(3, 1, 8, 16, 3)
    _, packed = gu.select_pack(w, 3, masks, 4, "bf16")
    _, wd, _ = gu.oracle_weights(w, 3, masks, 4, "bf16")
    ref = gu.oracle_conv(3, x, wd, None, 1, "relu", "bf16")
    for layout in ("nchw", "nhwc"):
        y = gu.run_conv(packed, 3, x, "bf16", 1, "relu", None, layout, y_off=5, y_stride=20)
        assert orc.rel_err(y[:, 5:13], ref) <= 2e-2
        assert (y[:, :5] == 7.0).all() and (y[:, 13:] == 7.0).all()
    packed.close()


def test_weights_given_in_16_bit_types():
    masks = _table(3)
    w = synth.kaiming_weights(4, 1, 24, 40, 3)
    for wdt in ("bf16", "f16"):
        pid_g, packed = gu.select_pack(w, 3, masks, 3, "bf16", w_dt=wdt)
        pid_o, _, arrays = gu.oracle_weights(w, 3, masks, 3, "bf16", w_dt=wdt)
        assert np.array_equal(pid_g, pid_o.ravel())
        ex = packed.export()
        assert np.array_equal(gu.val_as_f32(ex["val"], "bf16").view(np.uint32), arrays["val"].view(np.uint32))
        packed.close()


def test_select_and_pack_whole_yolov5s_stack_bit_exact():
    """Every layer of the YOLOv5s-shaped stack: ids, values, order arrays."""
    masks = _table(4)
    for li, L in enumerate(synth.yolov5s_stack()):
        w = synth.kaiming_weights(0, 1000 + li, L["cout"], L["cin"], L["ksize"])
        pid_g, packed = gu.select_pack(w, L["ksize"], masks, 4, "bf16")
        pid_o, wd, arrays = gu.oracle_weights(w, L["ksize"], masks, 4, "bf16")
        assert np.array_equal(pid_g, pid_o.ravel()), L["name"]
        ex = packed.export()
        assert np.array_equal(gu.val_as_f32(ex["val"], "bf16").view(np.uint32), arrays["val"].view(np.uint32))
        if L["ksize"] == 3:
            assert np.array_equal(ex["perm"], arrays["perm"]) and np.array_equal(ex["bucket_off"], arrays["bucket_off"])
        dense = packed.to_dense().float().cpu().numpy().reshape(wd.shape)
        assert np.array_equal(dense.view(np.uint32), wd.view(np.uint32))
        packed.close()


def test_select_special_values_match_oracle():
    masks = orc.pattern_preset(2, orc.PRESET_CONN4)
    w = synth.normal(6, 1, (64, 9)).copy()
    w[0] = 0.0
    w[1] = 1.0                       # all equal: tie -> lowest id
    w[2, 0] = np.nan
    w[3] = np.nan
    w[4] = 1e-30                     # squares are subnormal in fp32
    w[5] = 3e19                      # squares overflow to inf
    w[6, :] = [1, 1, 0, 0, 0, 0, 0, 1, 1]
    wd = torch.from_numpy(w.reshape(64, 1, 3, 3)).cuda()
    pid = gu.ctx().rtoss_select_patterns(wd, 3, masks, 2).cpu().numpy()
    assert np.array_equal(pid, orc.select_kernels(w, masks))


def test_dense_table_agrees_with_library_convolution():
    """k = 9 reduces to an ordinary convolution: compare with torch's own conv2d on the GPU."""
    masks = _table(9)
    x = synth.activations(7, 1, 2, 24, 30, 30)
    w = synth.kaiming_weights(7, 1, 40, 24, 3)
    _, packed = gu.select_pack(w, 3, masks, 9, "f32")
    for s in (1, 2):
        y = gu.run_conv(packed, 3, x, "f32", s, "none", None)
        ref = torch.nn.functional.conv2d(torch.from_numpy(x).double(), torch.from_numpy(w).double(), stride=s, padding=1)
        assert orc.rel_err(y, ref.numpy()) <= 1e-4
    packed.close()


def test_repeat_runs_are_bitwise_identical():
    masks = _table(3)
    x = synth.round_like(synth.activations(8, 1, 2, 64, 40, 40), "bf16")
    w = synth.kaiming_weights(8, 1, 64, 64, 3)
    _, packed = gu.select_pack(w, 3, masks, 3, "bf16")
    y1 = gu.run_conv(packed, 3, x, "bf16", 1, "silu", None)
    y2 = gu.run_conv(packed, 3, x, "bf16", 1, "silu", None)
    assert np.array_equal(y1.view(np.uint32), y2.view(np.uint32))
    packed.close()


@pytest.mark.parametrize("ksize", [3, 1])
def test_host_buffer_entry_point(ksize):
    gu.check_layer(9, 300 + ksize, ksize, 2, 32, 48, 20, 24, 1, 4, _table(4), "bf16", "silu", host=True)


def test_host_buffer_entry_point_chunked_batch():
    """A batch large enough to be cut into overlapping chunks (uneven: 7 images), both layouts, and a channel slice."""
    gu.check_layer(9, 310, 3, 7, 64, 64, 48, 40, 1, 4, _table(4), "bf16", "relu", layout="nhwc", host=True)
    gu.check_layer(9, 311, 1, 7, 64, 96, 48, 40, 2, 3, _table(3), "f32", "silu", layout="nchw", host=True)
    masks = _table(4)
    x = synth.round_like(synth.activations(9, 312, 6, 32, 40, 40), "bf16")
    w = synth.kaiming_weights(9, 312, 48, 32, 3)
    _, packed = gu.select_pack(w, 3, masks, 4, "bf16")
    _, wd, _ = gu.oracle_weights(w, 3, masks, 4, "bf16")
    y = gu.run_conv(packed, 3, x, "bf16", 1, "none", None, "nhwc", y_off=8, y_stride=64, host=True)
    ref = gu.oracle_conv(3, x, wd, None, 1, "none", "bf16")
    assert orc.rel_err(y[:, 8:56], ref) <= 2e-2
    assert (y[:, :8] == 7.0).all() and (y[:, 56:] == 7.0).all()
    packed.close()


def test_argument_errors_return_status_codes():
    c = gu.ctx()
    masks = _table(4)
    w = torch.zeros(8, 8, 3, 3, device="cuda")
    with pytest.raises(rt.RtossError) as e:
        c.rtoss_select_patterns(w, 3, [0x01B, 0x01B], 4)
    assert e.value.status == 2
    with pytest.raises(rt.RtossError) as e:
        c.rtoss_select_patterns(w, 5, masks, 4)
    assert e.value.status == 1
    mis = torch.zeros(8 * 8 * 9 + 1, device="cuda")[1:].view(8, 8, 3, 3)     # 4-byte offset: not 16-byte aligned
    with pytest.raises(rt.RtossError) as e:
        c.rtoss_select_patterns(mis, 3, masks, 4)
    assert e.value.status == 4
    pid = c.rtoss_select_patterns(w, 3, masks, 4)
    packed = c.rtoss_pack(w, 3, masks, 4, pid, rt.F32)
    x = torch.zeros(1, 8, 6, 6, device="cuda")
    y = torch.zeros(1, 8, 6, 6, device="cuda")
    with pytest.raises(rt.RtossError) as e:
        c.rtoss_conv1x1_pattern(packed, x, y, 1, 6, 6)                        # 3x3 handle given to the 1x1 call
    assert e.value.status == 1
    with pytest.raises(rt.RtossError) as e:
        c.rtoss_conv3x3_pattern(packed, x, y, 1, 6, 6, stride=3)
    assert e.value.status == 1
    with pytest.raises(rt.RtossError) as e:
        c.rtoss_conv3x3_pattern(packed, x, y, 1, 6, 6, y_channel_offset=4, y_channel_stride=8)
    assert e.value.status == 1
    c.rtoss_conv3x3_pattern(packed, x, y, 1, 6, 6)                            # the context stays usable
    torch.cuda.synchronize()
    packed.close()


def test_children_inherit_the_parent_layers_patterns():
    """Layer grouping (Algorithm 1) lets the layers of a group share kernel patterns: a child is packed with its
    PARENT's pattern ids (same shape, identity mapping of (co, ci)) instead of being re-selected."""
    masks = _table(3)
    nodes = [dict(kind="conv", cin=24, cout=24, ksize=3, inputs=[]), dict(kind="conv", cin=24, cout=24, ksize=3, inputs=[0]),
             dict(kind="op", inputs=[0, 1]), dict(kind="conv", cin=24, cout=24, ksize=3, inputs=[2])]
    parent, group, ng = rt.rtoss_group_layers(nodes)
    assert ng == 1 and parent.tolist() == [0, 0, -1, 0]
    c = gu.ctx()
    w_parent = synth.kaiming_weights(50, 1, 24, 24, 3)
    pid_parent = c.rtoss_select_patterns(torch.from_numpy(w_parent).cuda(), 3, masks, 3)
    pid_o = orc.select_3x3(w_parent, masks)
    assert np.array_equal(pid_parent.cpu().numpy(), pid_o.ravel())
    for child in (1, 3):
        w_child = synth.kaiming_weights(50, 1 + child, 24, 24, 3)
        packed = c.rtoss_pack(torch.from_numpy(w_child).cuda(), 3, masks, 3, pid_parent, rt.F32)
        dense = packed.to_dense().cpu().numpy()
        assert np.array_equal(dense, orc.mask_3x3(w_child, masks, pid_o))          # the parent's masks on the child's weights
        x = synth.activations(50, 9, 1, 24, 10, 10)
        y = gu.run_conv(packed, 3, x, "f32", 1, "none", None)
        assert orc.rel_err(y, gu.oracle_conv(3, x, dense, None, 1, "none", "f32")) <= 1e-4
        packed.close()


@pytest.mark.parametrize("k", [2, 3])
def test_pattern_usage_counts_match_oracle(k):
    """Criterion 2 of Section IV.B: win counts of every candidate pattern over a seeded sample of random kernels in
    [-1, 1); the oracle is its selection followed by a plain count.  Counts are integers: exact."""
    masks = orc.pattern_preset(k, orc.PRESET_CONN4)
    sample = synth.uniform_kernels(5, 1 << 18)
    counts = gu.ctx().rtoss_pattern_usage(torch.from_numpy(sample).cuda(), masks, k)
    want = np.bincount(orc.select_kernels(sample, masks), minlength=len(masks)).astype(np.uint64)
    assert np.array_equal(counts, want)
    assert int(counts.sum()) == sample.shape[0]
    assert (counts > 0).all()            # every edge-connected pattern wins somewhere in a quarter million kernels


@pytest.mark.parametrize("k,preset,M", [(3, "conn4", 8), (2, "conn4", 12), (4, "all", 21), (5, "conn4", 16)])
def test_pattern_table_derivation_matches_oracle(k, preset, M):
    """Section IV.B end to end: candidates from Eq. 1 (with or without the adjacency criterion), usage over a seeded
    sample in [-1, 1), the M most used.  Integers throughout: candidate table, counts and kept table are exact."""
    pre_g = {"conn4": rt.PRESET_CONN4, "all": rt.PRESET_ALL}[preset]
    pre_o = {"conn4": orc.PRESET_CONN4, "all": orc.PRESET_ALL}[preset]
    sample = synth.uniform_kernels(6, 1 << 17)
    top, cand, counts = gu.ctx().rtoss_pattern_table_derive(torch.from_numpy(sample).cuda(), k, pre_g, M)
    want_top, want_cand, want_counts = orc.derive_pattern_table(sample, k, pre_o, M)
    assert np.array_equal(cand, want_cand)
    assert np.array_equal(counts, want_counts)
    assert np.array_equal(top, want_top)
    assert rt.rtoss_pattern_table_validate(top, k) == rt.OK
    # the derived table is usable by the next step of the path
    w = synth.kaiming_weights(6, 2, 16, 8, 3)
    pid = gu.ctx().rtoss_select_patterns(torch.from_numpy(w).cuda(), 3, top, k)
    assert np.array_equal(pid.cpu().numpy().ravel(), orc.select_3x3(w, want_top).ravel())


def test_pack_with_ids_outside_the_table_stays_inside_its_arrays():
    """rtoss_pack's precondition is pid < P.  Ids that break it (here: ids chosen with a larger table) must not make the
    ordering pass write outside the channel's slice of perm: the other channels' slices and bucket offsets equal the
    oracle's, the offending filters are simply not listed, and the device reports no fault."""
    c = gu.ctx()
    masks = orc.pattern_preset(3, orc.PRESET_CONN4)[:6]          # P = 6
    Cout, Cin = 40, 24
    w = synth.kaiming_weights(51, 1, Cout, Cin, 3)
    pid_o = orc.select_3x3(w, masks)
    bad = pid_o.copy()
    bad[5, Cin - 1] = 9        # the last channel: the out-of-range slot would lie behind the end of perm
    bad[17, Cin - 1] = 200
    bad[3, 2] = 6              # an inner channel: the slot would lie in the next channel's slice
    wd = torch.from_numpy(w).cuda()
    packed = c.rtoss_pack(wd, 3, masks, 3, torch.from_numpy(bad).cuda().reshape(-1), rt.F32)
    torch.cuda.synchronize()
    ex = packed.export()
    _, perm_o, off_o = orc.pack_3x3(w, masks, 3, pid_o, orc.DT_F32)
    perm, off = ex["perm"].reshape(Cin, Cout), ex["bucket_off"].reshape(Cin, len(masks) + 1)
    perm_o, off_o = perm_o.reshape(Cin, Cout), off_o.reshape(Cin, len(masks) + 1)
    untouched = [ci for ci in range(Cin) if ci not in (2, Cin - 1)]
    assert np.array_equal(perm[untouched], perm_o[untouched]) and np.array_equal(off[untouched], off_o[untouched])
    for ci, dropped in ((2, {3}), (Cin - 1, {5, 17})):
        n_ok = Cout - len(dropped)
        listed = perm[ci][:n_ok]
        assert sorted(listed.tolist()) == sorted(set(range(Cout)) - dropped)
        assert off[ci][-1] == Cout and np.all(np.diff(off[ci][:-1].astype(np.int64)) >= 0)
    assert c.rtoss_device_status() == 0
    packed.close()


FINE_SHAPE = [
    # N, Cin, Cout, H, W, stride, dt   -- layers small enough for the FMA path's finer kernel shape (four pixels per lane)
    (1, 64, 64, 40, 40, 1, "bf16"),     # five lane columns: tiles 40 bytes apart, 8-byte activation vectors
    (1, 32, 32, 32, 32, 1, "f32"),      # the 32-channel fp32 test layer
    (1, 64, 48, 20, 20, 2, "f16"),
    (2, 40, 24, 13, 16, 1, "bf16"),
    (1, 128, 64, 25, 36, 2, "f32"),
]


@pytest.mark.parametrize("N,Cin,Cout,H,W,stride,dt", FINE_SHAPE)
def test_fma_path_finer_shape_small_nchw_layers(N, Cin, Cout, H, W, stride, dt):
    """The shape's staging plan is checked vector by vector on the host (test_fma_plan_cpu.py); here its results."""
    p = rt.rtoss_fma_plan3x3(N, H, W, stride, rt.NCHW, rt.DTYPE_NAMES[dt], Cin, Cout, 4)
    assert p.pixels_per_lane == 4
    masks = orc.pattern_preset(4, orc.PRESET_CENTRE8)
    gu.check_layer(52, Cin + Cout + H, 3, N, Cin, Cout, H, W, stride, 4, masks, dt, "silu", "nchw", path=rt.PATH_FMA)
    assert gu.ctx().rtoss_device_status() == 0
