"""GPU parity of (a) the block-shared pattern selection and the tensor path's skipping of all-pruned blocks that it
enables, (b) several convolutions in one launch (rtoss_conv_group), (c) the bounded device waits running out on a
withheld copy.  Everything is compared with the CPU oracle on the same seeded inputs, through the C ABI."""
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


SHARED_SELECT = [
    # Cout, Cin, FB, CB, k, dtype
    (256, 256, 128, 16, 4, "f32"),
    (130, 72, 128, 16, 3, "f32"),      # ragged filter and channel blocks
    (64, 48, 64, 8, 2, "bf16"),
    (40, 36, 16, 8, 4, "f16"),
    (11, 10, 1, 1, 4, "f32"),          # blocks of one kernel
    (200, 24, 256, 24, 4, "f32"),      # one block over all filters
]


@pytest.mark.parametrize("Cout,Cin,FB,CB,k,dt", SHARED_SELECT)
def test_shared_selection_ids_bit_exact(Cout, Cin, FB, CB, k, dt):
    masks = _table(k)
    w = synth.round_like(synth.kaiming_weights(71, Cout * 7 + Cin, Cout, Cin, 3), dt)
    want = orc.select_shared(w, masks, FB, CB)
    got = gu.ctx().rtoss_select_patterns_shared(gu.to_dev(w, dt), masks, k, FB, CB)
    torch.cuda.synchronize()
    assert np.array_equal(got.cpu().numpy().reshape(Cout, Cin), want)


def _shared_layer(seed, tid, N, Cin, Cout, H, W, stride, k, dt, act, FB=128, CB=16, y_off=0, y_stride=0):
    """A 3x3 layer pruned with block-shared patterns: ids, packed arrays and outputs against the oracle."""
    c = gu.ctx()
    masks = _table(k)
    x = synth.round_like(synth.activations(seed, tid, N, Cin, H, W), dt)
    w = synth.kaiming_weights(seed, tid, Cout, Cin, 3)
    b = synth.bias(seed, tid, Cout)
    wd = gu.to_dev(w, "f32")
    pid = c.rtoss_select_patterns_shared(wd, masks, k, FB, CB)
    pid_o = orc.select_shared(w, masks, FB, CB)
    assert np.array_equal(pid.cpu().numpy().reshape(Cout, Cin), pid_o)
    packed = c.rtoss_pack(wd, 3, masks, k, pid, rt.DTYPE_NAMES[dt])
    val, perm, off = orc.pack_3x3(w, masks, k, pid_o, gu.ORC_DT[dt])
    ex = packed.export()
    assert np.array_equal(gu.val_as_f32(ex["val"], dt).view(np.uint32), val.view(np.uint32))
    assert np.array_equal(ex["perm"], perm) and np.array_equal(ex["bucket_off"], off)
    wdense = orc.unpack_3x3(val, Cout, Cin, masks, k, pid_o)
    y = gu.run_conv(packed, 3, x, dt, stride, act, b, "nhwc", y_off=y_off, y_stride=y_stride, path=rt.PATH_TENSOR)
    ref = gu.oracle_conv(3, x, wdense, b, stride, act, dt)
    if y_stride:
        assert np.all(y[:, :y_off] == 7.0) and np.all(y[:, y_off + Cout:] == 7.0)
        y = y[:, y_off:y_off + Cout]
    err = orc.rel_err(y, ref)
    assert err <= gu.TOL[dt], err
    return packed, w, masks, x, b


SHARED_CONV = [
    # N, Cin, Cout, H, W, stride, k, dt, act
    (1, 256, 256, 20, 20, 1, 4, "bf16", "silu"),     # two filter tiles, four channel blocks: 4 of 9 taps issued per slab
    (2, 128, 128, 40, 40, 1, 3, "bf16", "relu"),
    (1, 72, 200, 13, 17, 1, 2, "f16", "none"),       # ragged channel block and filter tile
    (1, 64, 64, 25, 34, 1, 4, "bf16", "silu"),       # narrow layer: filters repeated down the tile's rows
    (1, 128, 256, 40, 40, 2, 4, "bf16", "silu"),     # stride 2: one tap per weight stage
    (1, 512, 512, 7, 9, 1, 4, "bf16", "relu"),       # few tiles, many channel blocks: cut along K through a cluster
]


@pytest.mark.parametrize("N,Cin,Cout,H,W,stride,k,dt,act", SHARED_CONV)
def test_convolution_over_block_shared_patterns(N, Cin, Cout, H, W, stride, k, dt, act):
    packed, *_ = _shared_layer(72, Cin + Cout + H, N, Cin, Cout, H, W, stride, k, dt, act)
    packed.close()
    assert gu.ctx().rtoss_device_status() == 0


def test_output_slice_and_coarser_blocks():
    packed, *_ = _shared_layer(73, 1, 1, 128, 128, 20, 20, 1, 4, "bf16", "silu", FB=128, CB=64, y_off=64, y_stride=256)
    packed.close()
    packed, *_ = _shared_layer(73, 2, 1, 96, 160, 16, 16, 1, 4, "bf16", "none", FB=32, CB=16)   # blocks finer than a filter tile
    packed.close()
    assert gu.ctx().rtoss_device_status() == 0


def test_repacking_a_handle_refreshes_what_is_skipped():
    """A handle first packed with shared patterns (most blocks skipped) and then re-packed in place with per-kernel
    patterns (nothing skipped), by rtoss_pack and by the whole-model pass, must multiply the new weights' taps."""
    c = gu.ctx()
    N, Cin, Cout, H, W, k, dt = 1, 128, 128, 16, 16, 4, "bf16"
    packed, w, masks, x, b = _shared_layer(74, 1, N, Cin, Cout, H, W, 1, k, dt, "none")
    wd = gu.to_dev(w, "f32")
    pid = c.rtoss_select_patterns(wd, 3, masks, k)
    c.rtoss_pack(wd, 3, masks, k, pid, rt.DTYPE_NAMES[dt], into=packed)
    pid_o, wdense, _ = gu.oracle_weights(w, 3, masks, k, dt)
    ref = gu.oracle_conv(3, x, wdense, b, 1, "none", dt)
    y = gu.run_conv(packed, 3, x, dt, 1, "none", b, "nhwc", path=rt.PATH_TENSOR)
    assert orc.rel_err(y, ref) <= gu.TOL[dt]
    # back to shared patterns, then the whole-model pass (per-kernel selection) over the same handle
    c.rtoss_pack(wd, 3, masks, k, c.rtoss_select_patterns_shared(wd, masks, k, 128, 16), rt.DTYPE_NAMES[dt], into=packed)
    batch = c.rtoss_batch_create([dict(w=wd, ksize=3, masks=masks, k=k, packed=packed, pid=None)])
    batch.rtoss_batch_select_pack()
    y = gu.run_conv(packed, 3, x, dt, 1, "none", b, "nhwc", path=rt.PATH_TENSOR)
    assert orc.rel_err(y, ref) <= gu.TOL[dt]
    torch.cuda.synchronize()
    batch.close()
    packed.close()
    assert c.rtoss_device_status() == 0


# ------------------------------------------------------------------------------------------- several convolutions, one launch

def _member(c, seed, tid, ks, N, Cin, Cout, H, W, stride, k, dt, act, packed=None, w=None, b=None, shared=False):
    masks = _table(k)
    x = synth.round_like(synth.activations(seed, 100 + tid, N, Cin, H, W), dt)
    if packed is None:
        w = synth.kaiming_weights(seed, tid, Cout, Cin, ks)
        b = synth.bias(seed, tid, Cout)
        wd = gu.to_dev(w, "f32")
        pid = c.rtoss_select_patterns_shared(wd, masks, k, 128, 16) if shared else c.rtoss_select_patterns(wd, ks, masks, k)
        packed = c.rtoss_pack(wd, ks, masks, k, pid, rt.DTYPE_NAMES[dt])
    if ks == 3:
        pid_o = orc.select_shared(w, masks, 128, 16) if shared else orc.select_3x3(w, masks)
        wdense = orc.unpack_3x3(orc.pack_3x3(w, masks, k, pid_o, gu.ORC_DT[dt])[0], Cout, Cin, masks, k, pid_o)
    else:
        w2 = w.reshape(Cout, Cin)
        pid_o = orc.select_1x1(w2, masks)
        wdense = orc.unpack_1x1(orc.pack_1x1(w2, masks, k, pid_o, gu.ORC_DT[dt]), Cout, Cin, masks, k, pid_o)
    ref = gu.oracle_conv(ks, x, wdense, b, stride, act, dt)
    return dict(ks=ks, N=N, H=H, W=W, stride=stride, act=act, packed=packed, w=w, b=b, x=x, ref=ref, dt=dt, Cout=Cout)


def _run_group(c, members, layout=None):
    items, outs = [], []
    for m in members:
        xd = gu.to_dev(m["x"], m["dt"], "nhwc")
        Ho, Wo = synth.out_hw(m["H"], m["W"], m["stride"])
        yd = torch.full((m["N"], Ho, Wo, m["Cout"]), 7.0, dtype=gu.TORCH_DT[m["dt"]], device="cuda")
        bd = torch.from_numpy(m["b"]).cuda()
        res = m.get("res")
        rd = gu.to_dev(res, m["dt"], "nhwc") if res is not None else None
        items.append(c.conv_item(m["packed"], xd, yd, m["N"], m["H"], m["W"], m["stride"], rt.NHWC, ACT[m["act"]], bd, residual=rd))
        outs.append((xd, yd, bd, rd))
    n = c.rtoss_conv_group(items)
    torch.cuda.synchronize()
    for m, (_, yd, _, _) in zip(members, outs):
        y = gu.from_dev(yd, "nhwc")
        err = orc.rel_err(y, m["ref"])
        assert err <= gu.TOL[m["dt"]], (m["H"], m["W"], err)
    return n


def test_one_tower_layer_over_five_pyramid_levels_in_one_launch():
    """The five levels share one weight tensor; the small levels ride in the large one's launch."""
    c = gu.ctx()
    first = _member(c, 75, 1, 3, 2, 256, 256, 50, 68, 1, 4, "bf16", "relu")
    members = [first]
    for i, (H, W) in enumerate([(25, 34), (13, 17), (7, 9), (4, 5)]):
        members.append(_member(c, 75, 2 + i, 3, 2, 256, 256, H, W, 1, 4, "bf16", "relu", packed=first["packed"], w=first["w"], b=first["b"]))
    assert _run_group(c, members) == 1
    assert _run_group(c, members[::-1]) == 1      # any order of the items
    first["packed"].close()
    assert c.rtoss_device_status() == 0


def test_two_towers_with_shared_patterns_and_different_weights():
    c = gu.ctx()
    a = _member(c, 76, 1, 3, 1, 128, 128, 30, 40, 1, 4, "bf16", "relu", shared=True)
    b = _member(c, 76, 2, 3, 1, 128, 256, 15, 20, 1, 4, "bf16", "silu", shared=True)
    d = _member(c, 76, 3, 3, 1, 64, 64, 9, 11, 1, 3, "bf16", "none")          # narrow: filters repeated down the rows
    assert _run_group(c, [a, b, d]) == 1
    for m in (a, b, d):
        m["packed"].close()
    assert c.rtoss_device_status() == 0


def test_1x1_branches_strides_residual_and_mixed_items():
    c = gu.ctx()
    a = _member(c, 77, 1, 1, 2, 256, 128, 20, 20, 1, 4, "bf16", "relu")
    b = _member(c, 77, 2, 1, 2, 256, 512, 20, 20, 2, 4, "bf16", "none")       # a stride-2 projection next to it
    b["res"] = synth.round_like(synth.activations(77, 50, 2, 512, 10, 10), "bf16")
    b["ref"] = orc.add_act(b["ref"], b["res"], orc.ACT_NONE, orc.DT_BF16)
    assert _run_group(c, [a, b]) == 1
    # items the shared launch does not take (few filters with the positions on M; a 3x3 among 1x1) run on their own
    n32 = _member(c, 77, 3, 1, 2, 64, 32, 20, 20, 1, 4, "bf16", "silu")
    k3 = _member(c, 77, 4, 3, 2, 64, 128, 20, 20, 1, 4, "bf16", "silu")
    del b["res"]
    b["ref"] = gu.oracle_conv(1, b["x"], *(_dense_1x1(b)), 2, "none", "bf16")
    assert _run_group(c, [a, n32, b, k3]) == 3
    assert _run_group(c, [n32]) == 1
    for m in (a, b, n32, k3):
        m["packed"].close()
    assert c.rtoss_device_status() == 0


def _dense_1x1(m):
    masks = _table(4)
    w2 = m["w"].reshape(m["Cout"], -1)
    pid = orc.select_1x1(w2, masks)
    return orc.unpack_1x1(orc.pack_1x1(w2, masks, 4, pid, orc.DT_BF16), m["Cout"], w2.shape[1], masks, 4, pid), m["b"]


def test_group_of_fp16_many_tiles():
    c = gu.ctx()
    ms = [_member(c, 78, i, 3, 3, 64, 128, H, W, 1, 3, "f16", "silu") for i, (H, W) in enumerate([(80, 80), (33, 47), (5, 300 // 2)])]
    assert _run_group(c, ms) == 1
    for m in ms:
        m["packed"].close()
    assert c.rtoss_device_status() == 0


# ------------------------------------------------------------------------------------------- a bounded wait that runs out

def test_withheld_copy_times_out_and_the_context_stays_usable():
    """Failure detection without a fault: the launch's first weight copy is withheld, the waits that depend on it give up
    after the (shortened) limit, the kernel ends normally and the status word reports it; the next call is right."""
    c = rt.Context(0)
    masks = _table(4)
    x = synth.round_like(synth.activations(79, 1, 1, 64, 8, 8), "bf16")
    w = synth.kaiming_weights(79, 1, 64, 64, 3)
    wd = gu.to_dev(w, "f32")
    pid = c.rtoss_select_patterns(wd, 3, masks, 4)
    packed = c.rtoss_pack(wd, 3, masks, 4, pid, rt.BF16)
    xd = gu.to_dev(x, "bf16", "nhwc")
    yd = torch.zeros(1, 8, 8, 64, dtype=torch.bfloat16, device="cuda")
    c.rtoss_set_wait_limit(200000)               # a tenth of a millisecond
    c.rtoss_inject_lost_copy()
    c.rtoss_conv3x3_pattern(packed, xd, yd, 1, 8, 8, 1, rt.NHWC, rt.ACT_NONE, None, path=rt.PATH_TENSOR)
    code = c.rtoss_device_status()
    assert code != 0                             # RTOSS_ERR_TIMEOUT was reported, with the code of the role that gave up
    assert c.rtoss_device_status() == 0          # reading it clears it
    c.rtoss_set_wait_limit(2000000000)
    c.rtoss_conv3x3_pattern(packed, xd, yd, 1, 8, 8, 1, rt.NHWC, rt.ACT_NONE, None, path=rt.PATH_TENSOR)
    assert c.rtoss_device_status() == 0
    _, wdense, _ = gu.oracle_weights(w, 3, masks, 4, "bf16")
    ref = gu.oracle_conv(3, x, wdense, None, 1, "none", "bf16")
    assert orc.rel_err(gu.from_dev(yd, "nhwc"), ref) <= 2e-2
    # a launch of more than one CTA does not take the request, and the request does not linger
    c.rtoss_inject_lost_copy()
    x2 = gu.to_dev(synth.round_like(synth.activations(79, 2, 4, 64, 40, 40), "bf16"), "bf16", "nhwc")
    y2 = torch.zeros(4, 40, 40, 64, dtype=torch.bfloat16, device="cuda")
    with pytest.raises(rt.RtossError):
        c.rtoss_conv3x3_pattern(packed, x2, y2, 4, 40, 40, 1, rt.NHWC, rt.ACT_NONE, None, path=rt.PATH_TENSOR)
    c.rtoss_conv3x3_pattern(packed, x2, y2, 4, 40, 40, 1, rt.NHWC, rt.ACT_NONE, None, path=rt.PATH_TENSOR)
    assert c.rtoss_device_status() == 0
    packed.close()
    c.close()
