"""Host logic of the tensor path's tile planner (rtoss_tensor_plan_of: plain arithmetic through the C ABI, no GPU):
the invariants the kernel and the TMA descriptors rely on, over the layer shapes of both model families and a sweep of
odd ones."""
import itertools

import pytest

from paper_2303_02191_b200 import binding as rt
from paper_2303_02191_b200 import synth

BF16, F16, F32 = rt.DTYPE_NAMES["bf16"], rt.DTYPE_NAMES["f16"], rt.DTYPE_NAMES["f32"]
CAP = 227 * 1024


def check(N, H, W, S, ks, Cin, Cout, dt, residual=False):
    p = rt.rtoss_tensor_plan_of(N, H, W, S, ks, Cin, Cout, dt, residual=residual)
    es = 4 if dt == F32 else 2
    if not p.eligible:
        return p
    Ho, Wo = synth.out_hw(H, W, S)
    halo = (2 if S == 1 else 1) if ks == 3 else 0
    assert p.shared_bytes <= CAP
    assert 16 <= p.positions <= 256 and p.positions % 16 == 0
    assert p.pitch == p.cols_per_tile + halo and p.rows_per_tile * p.pitch <= p.positions
    assert p.staged_rows == p.rows_per_tile + halo
    # a TMA box traverses at most 256 elements per dimension (stride-2 boxes traverse every second one)
    assert p.pitch * S <= 256 and p.staged_rows * S <= 256
    assert p.row_bytes == (64 if (dt != F32 and Cin <= 32) else 128)
    # stage sizes are multiples of the swizzle atom (8 rows), so every stage starts on an atom boundary
    assert p.act_stage_bytes % (8 * p.row_bytes) == 0 and p.weight_stage_bytes % (8 * p.row_bytes) == 0
    assert p.sub_tiles == (4 if (ks == 3 and S == 2) else 1)
    assert 1 <= p.act_stages <= 4 and 2 <= p.weight_stages <= 8
    assert p.taps_per_weight_stage in ((1, 3) if ks == 3 else (1,))
    assert p.act_stages * p.act_stage_bytes + p.weight_stages * p.weight_stage_bytes < p.shared_bytes
    # the tiles cover the output
    tiles_y = -(-Ho // p.rows_per_tile)
    tiles_x = -(-Wo // p.cols_per_tile)
    co_tiles = 1 if p.positions_on_m else -(-Cout // 128)
    assert p.tiles == N * tiles_y * tiles_x * co_tiles
    assert p.positions_on_m == (1 if (ks == 1 and Cout <= 64 and dt != F32) else 0)
    cb_ch = p.row_bytes // es
    ncb = -(-Cin // cb_ch)
    assert 1 <= p.split_k <= min(8, ncb)
    if p.split_k > 1:
        assert p.tiles * 2 <= 148 and not p.positions_on_m
    return p


def test_every_layer_of_both_model_families():
    for N, layers in ((16, synth.yolov5s_stack()), (1, synth.yolov5s_stack()), (4, synth.retinanet_r50fpn_stack())):
        for L in layers:
            if L["cin"] % 8:
                continue
            p = check(N, L["H"], L["W"], L["stride"], L["ksize"], L["cin"], L["cout"], BF16)
            assert p.eligible, L["name"]


def test_odd_shapes_and_types():
    for (H, W), S, ks, (Cin, Cout), dt in itertools.product(
            [(1, 1), (7, 9), (13, 255), (64, 64), (5, 700), (200, 272), (3, 2000)], (1, 2), (1, 3),
            [(8, 8), (24, 20), (32, 32), (40, 80), (64, 48), (72, 200), (256, 256), (2048, 512)], (BF16, F16, F32)):
        check(2, H, W, S, ks, Cin, Cout, dt)
        check(1, H, W, S, ks, Cin, Cout, dt, residual=True)


def test_ineligible_shapes_and_bad_arguments():
    assert not rt.rtoss_tensor_plan_of(1, 8, 8, 1, 3, 12, 16, BF16).eligible      # rows of 24 bytes: not a multiple of 16
    assert not rt.rtoss_tensor_plan_of(1, 8, 8, 1, 3, 6, 16, F32).eligible
    assert not rt.rtoss_tensor_plan_of(1, 8, 8, 1, 3, 64, 64, BF16, layout=rt.NCHW).eligible
    for bad in ((0, 8, 8, 1, 3, 64, 64), (1, 8, 8, 3, 3, 64, 64), (1, 8, 8, 1, 2, 64, 64), (1, 8, 8, 1, 3, 0, 64)):
        with pytest.raises(rt.RtossError):
            rt.rtoss_tensor_plan_of(*bad, BF16)


def test_narrow_layers_stage_half_rows_and_keep_a_deeper_ring():
    p = check(16, 160, 160, 1, 3, 32, 32, BF16)
    assert p.row_bytes == 64 and p.act_stages > 2        # one channel block per tile: the next tile's block is the next stage
    q = check(16, 160, 160, 1, 3, 128, 128, BF16)
    assert q.row_bytes == 128 and q.act_stages == 2
