"""Whole-model pruning pass (selection + packing of every layer in two launches) against the CPU oracle,
layer by layer and bit for bit; inheritance of a parent's patterns; the convolution after a batch re-pack."""
import numpy as np
import pytest
import torch

from oracle import rtoss_oracle as orc
from paper_2303_02191_b200 import binding as rt
from paper_2303_02191_b200 import synth
from gpu_util import ORC_DT, TOL, ctx, from_dev, oracle_weights, to_dev, val_as_f32

pytestmark = pytest.mark.gpu

# (Cout, Cin, ksize, k, preset, w dtype): several chunks and ragged tails, a 1x1 with leftovers, a 1x1 with no full
# run of nine, narrow and wide layers, every storage type
LAYERS = [
    (32, 3, 3, 4, rt.PRESET_CENTRE8, "f32"),
    (64, 32, 3, 3, rt.PRESET_CONN4, "f32"),
    (40, 24, 1, 4, rt.PRESET_CENTRE8, "f32"),     # 960 weights: 106 runs, 6 left over
    (2, 3, 1, 4, rt.PRESET_CENTRE8, "f32"),       # 6 weights: no run at all
    (128, 128, 3, 2, rt.PRESET_CONN4, "bf16"),
    (256, 128, 1, 3, rt.PRESET_CONN4, "f16"),
    (96, 48, 3, 9, rt.PRESET_DENSE, "f32"),
    (130, 33, 3, 5, rt.PRESET_ALL, "f32"),        # 4290 kernels: 16 full chunks + a tail of 194; P = 126
]


def _make(seed, compute_dt, layers=LAYERS):
    c = ctx()
    made = []
    for i, (co, ci, ks, k, preset, wdt) in enumerate(layers):
        masks = rt.rtoss_pattern_preset(k, preset)
        w = synth.round_like(synth.kaiming_weights(seed, 300 + i, co, ci, ks), wdt)
        wd = to_dev(w, wdt)
        pid = c.rtoss_select_patterns(wd, ks, masks, k)
        packed = c.rtoss_pack(wd, ks, masks, k, pid, rt.DTYPE_NAMES[compute_dt])
        made.append(dict(w=wd, w_np=w, ksize=ks, masks=masks, k=k, packed=packed, pid=torch.zeros_like(pid), wdt=wdt))
    torch.cuda.synchronize()
    return made


def _check_layer(L, w_np, compute_dt, pid_expect=None):
    co, ci = w_np.shape[0], w_np.shape[1]
    pid_o, wd_o, arrays = oracle_weights(w_np, L["ksize"], L["masks"], L["k"], compute_dt, L["wdt"])
    if pid_expect is not None:
        pid_o = pid_expect
        if L["ksize"] == 3:
            val, perm, off = orc.pack_3x3(w_np, L["masks"], L["k"], pid_o, ORC_DT[compute_dt])
            arrays = dict(val=val, perm=perm, bucket_off=off)
            wd_o = orc.unpack_3x3(val, co, ci, L["masks"], L["k"], pid_o)
        else:
            val = orc.pack_1x1(w_np.reshape(co, ci), L["masks"], L["k"], pid_o, ORC_DT[compute_dt])
            arrays = dict(val=val)
            wd_o = orc.unpack_1x1(val, co, ci, L["masks"], L["k"], pid_o)
    n = pid_o.size
    ex = L["packed"].export()
    assert np.array_equal(L["pid"].cpu().numpy().ravel()[:n], pid_o.ravel())
    assert np.array_equal(ex["pid"][:n], pid_o.ravel())
    got_val = val_as_f32(ex["val"], compute_dt)[: n * L["k"]]
    assert np.array_equal(got_val.view(np.uint32), np.asarray(arrays["val"], dtype=np.float32).ravel()[: n * L["k"]].view(np.uint32))
    if L["ksize"] == 3:
        assert np.array_equal(ex["perm"][: ci * co], np.asarray(arrays["perm"]).ravel())
        assert np.array_equal(ex["bucket_off"][: ci * (len(L["masks"]) + 1)], np.asarray(arrays["bucket_off"]).ravel())
    dense = from_dev(L["packed"].to_dense())
    assert np.array_equal(dense.ravel().view(np.uint32), np.asarray(wd_o, dtype=np.float32).ravel().view(np.uint32))
    return pid_o


@pytest.mark.parametrize("compute_dt", ["f32", "bf16"])
def test_batch_matches_oracle_after_weight_update(compute_dt):
    c = ctx()
    made = _make(1, compute_dt)
    batch = c.rtoss_batch_create(made)
    # the weights change (one step of the iterative loop), then ONE pass re-selects and re-packs every layer
    for i, L in enumerate(made):
        co, ci = L["w_np"].shape[:2]
        L["w_np"] = synth.round_like(synth.kaiming_weights(2, 900 + i, co, ci, L["ksize"]), L["wdt"])
        L["w"].copy_(to_dev(L["w_np"], L["wdt"]))
    batch.rtoss_batch_select_pack()
    batch.rtoss_batch_select_pack()   # a second pass over unchanged weights changes nothing
    torch.cuda.synchronize()
    for L in made:
        _check_layer(L, L["w_np"], compute_dt)
    assert c.rtoss_device_status() == 0
    batch.close()
    for L in made:
        L["packed"].close()


def test_batch_inherits_parent_patterns():
    """Children of a group take the parent's pattern ids (also through a chain) and keep their own values."""
    c = ctx()
    layers = [(64, 64, 3, 4, rt.PRESET_CENTRE8, "f32")] * 3 + [(72, 18, 1, 3, rt.PRESET_CONN4, "bf16")] * 2
    made = _make(3, "bf16", layers)
    made[1]["pid_from"] = 0
    made[2]["pid_from"] = 1          # chain: the root is layer 0
    made[4]["pid_from"] = 3
    batch = c.rtoss_batch_create(made)
    batch.rtoss_batch_select_pack()
    torch.cuda.synchronize()
    root = _check_layer(made[0], made[0]["w_np"], "bf16")
    _check_layer(made[1], made[1]["w_np"], "bf16", pid_expect=root)
    _check_layer(made[2], made[2]["w_np"], "bf16", pid_expect=root)
    root1 = _check_layer(made[3], made[3]["w_np"], "bf16")
    _check_layer(made[4], made[4]["w_np"], "bf16", pid_expect=root1)
    # and the ids differ from what the children would have chosen for themselves
    own = orc.select_3x3(made[1]["w_np"], made[1]["masks"])
    assert (own != root).any()
    batch.close()
    for L in made:
        L["packed"].close()


def test_conv_after_batch_repack_tensor_path():
    """The tensor path's dense-expanded weights are rebuilt by the batch: convolution parity after a re-pack."""
    c = ctx()
    layers = [(128, 64, 3, 3, rt.PRESET_CONN4, "f32"), (128, 128, 1, 4, rt.PRESET_CENTRE8, "f32")]
    made = _make(5, "bf16", layers)
    batch = c.rtoss_batch_create(made)
    for i, L in enumerate(made):
        co, ci = L["w_np"].shape[:2]
        L["w_np"] = synth.kaiming_weights(6, 40 + i, co, ci, L["ksize"])
        L["w"].copy_(to_dev(L["w_np"], "f32"))
    batch.rtoss_batch_select_pack()
    N, H, W = 2, 20, 24
    for i, L in enumerate(made):
        co, ci = L["w_np"].shape[:2]
        x = synth.round_like(synth.activations(6, 70 + i, N, ci, H, W), "bf16")
        b = synth.bias(6, 80 + i, co)
        xd = to_dev(x, "bf16", "nhwc")
        y = torch.empty((N, H, W, co), dtype=torch.bfloat16, device="cuda")
        fn = c.rtoss_conv3x3_pattern if L["ksize"] == 3 else c.rtoss_conv1x1_pattern
        fn(L["packed"], xd, y, N, H, W, 1, rt.NHWC, rt.ACT_SILU, torch.from_numpy(b).cuda(), path=rt.PATH_TENSOR)
        _, wd_o, _ = oracle_weights(L["w_np"], L["ksize"], L["masks"], L["k"], "bf16")
        conv = orc.conv3x3 if L["ksize"] == 3 else orc.conv1x1
        ref = conv(x, wd_o, b, 1, orc.ACT_SILU, ORC_DT["bf16"])
        assert orc.rel_err(from_dev(y, "nhwc"), ref) <= TOL["bf16"]
    assert c.rtoss_device_status() == 0
    batch.close()
    for L in made:
        L["packed"].close()


def test_batch_rejects_bad_items():
    c = ctx()
    made = _make(7, "f32", LAYERS[:2])
    with pytest.raises(rt.RtossError) as e:
        c.rtoss_batch_create([made[0], made[0]])          # one handle twice
    assert e.value.status == 1
    bad = dict(made[1]); bad["pid_from"] = 0              # another shape
    with pytest.raises(rt.RtossError) as e:
        c.rtoss_batch_create([made[0], bad])
    assert e.value.status == 1
    bad = dict(made[0]); bad["pid_from"] = 0              # not an EARLIER item
    with pytest.raises(rt.RtossError) as e:
        c.rtoss_batch_create([bad])
    assert e.value.status == 1
    bad = dict(made[0]); bad["masks"] = np.array([7, 7], dtype=np.uint16)
    with pytest.raises(rt.RtossError):
        c.rtoss_batch_create([bad])
    for L in made:
        L["packed"].close()
