"""GPU parity of the tensor-core path (tcgen05 masked dense implicit GEMM, bf16 / fp16 NHWC) against
the CPU oracle, and agreement with the FMA path on the same inputs."""
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


def _no_timeout():
    assert gu.ctx().rtoss_device_status() == 0, "a device-side wait of the tensor path ran out"


def test_tensor_path_smallest_case():
    """One CTA, one channel block: the first thing to run after any change to the kernel."""
    gu.check_layer(20, 1, 3, 1, 64, 64, 8, 8, 1, 4, _table(4), "bf16", "none", "nhwc", use_bias=False, path=rt.PATH_TENSOR)
    _no_timeout()


CASES = [
    # ksize, N, Cin, Cout, H, W, k, dt, act   (stride 1)
    (3, 1, 128, 128, 80, 80, 3, "bf16", "silu"),      # the 128-channel layer, one image
    (3, 2, 64, 64, 40, 40, 4, "bf16", "silu"),
    (3, 1, 32, 64, 20, 20, 4, "bf16", "relu"),        # half-filled channel block
    (3, 1, 72, 48, 13, 17, 2, "f16", "none"),         # ragged channel block, N_T not a multiple of 32, odd size
    (3, 1, 256, 256, 20, 20, 4, "bf16", "silu"),      # two filter tiles
    (3, 1, 64, 512, 7, 9, 4, "bf16", "relu"),         # four filter tiles, tiny image
    (3, 2, 128, 16, 25, 34, 9, "bf16", "none"),       # dense table, narrow N
    (3, 1, 64, 64, 1, 1, 4, "bf16", "none"),          # single pixel
    (3, 1, 64, 32, 3, 200, 3, "f16", "silu"),         # wide image
    (1, 1, 256, 128, 80, 80, 3, "bf16", "silu"),      # the 256->128 1x1 layer, one image
    (1, 2, 64, 32, 20, 20, 4, "bf16", "silu"),
    (1, 1, 1024, 512, 20, 20, 4, "bf16", "silu"),
    (1, 1, 40, 80, 13, 17, 2, "f16", "relu"),
    (1, 1, 512, 2048, 25, 34, 4, "bf16", "relu"),
    (3, 1, 24, 20, 9, 11, 3, "bf16", "silu"),         # filter count not a multiple of 16, 24 channels
    (1, 3, 8, 200, 5, 254, 2, "f16", "none"),         # widest image the path takes, filter tiles 128 + 72
]


STRIDED_AND_WIDE = [
    # ksize, stride, N, Cin, Cout, H, W, k, dt, act
    (3, 2, 1, 64, 128, 40, 40, 4, "bf16", "silu"),     # downsampling conv, even size
    (3, 2, 2, 128, 128, 25, 34, 4, "bf16", "relu"),    # odd height
    (3, 2, 1, 32, 64, 13, 17, 3, "f16", "none"),       # both odd
    (3, 2, 1, 72, 40, 9, 250, 2, "bf16", "silu"),      # wide, stride 2: column segments
    (3, 2, 1, 256, 256, 2, 2, 4, "bf16", "none"),      # one output pixel
    (1, 2, 1, 256, 512, 50, 68, 4, "bf16", "none"),    # strided 1x1 (downsample branch)
    (1, 2, 2, 64, 32, 7, 9, 3, "f16", "relu"),
    (3, 1, 1, 64, 64, 10, 272, 4, "bf16", "relu"),     # wider than one TMA box: column segments
    (1, 1, 1, 64, 256, 6, 300, 4, "bf16", "relu"),
    (3, 1, 1, 16, 24, 5, 700, 3, "f16", "silu"),
]


@pytest.mark.parametrize("case", STRIDED_AND_WIDE, ids=lambda c: "-".join(str(v) for v in c))
def test_tensor_path_strided_and_wide(case):
    ks, s, N, Cin, Cout, H, W, k, dt, act = case
    gu.check_layer(25, 700 + Cin + W, ks, N, Cin, Cout, H, W, s, k, _table(k), dt, act, "nhwc", path=rt.PATH_TENSOR)
    _no_timeout()


@pytest.mark.parametrize("case", CASES, ids=lambda c: "-".join(str(v) for v in c))
def test_tensor_path_against_oracle(case):
    ks, N, Cin, Cout, H, W, k, dt, act = case
    gu.check_layer(21, 400 + Cin + Cout, ks, N, Cin, Cout, H, W, 1, k, _table(k), dt, act, "nhwc", path=rt.PATH_TENSOR)
    _no_timeout()


@pytest.mark.parametrize("ksize", [3, 1])
def test_tensor_and_fma_paths_agree(ksize):
    masks = _table(4)
    N, Cin, Cout, H, W = 2, 128, 128, 30, 30
    x = synth.round_like(synth.activations(22, ksize, N, Cin, H, W), "bf16")
    w = synth.kaiming_weights(22, ksize, Cout, Cin, ksize)
    b = synth.bias(22, ksize, Cout)
    _, packed = gu.select_pack(w, ksize, masks, 4, "bf16")
    y_t = gu.run_conv(packed, ksize, x, "bf16", 1, "silu", b, "nhwc", path=rt.PATH_TENSOR)
    y_f = gu.run_conv(packed, ksize, x, "bf16", 1, "silu", b, "nhwc", path=rt.PATH_FMA)
    y_a = gu.run_conv(packed, ksize, x, "bf16", 1, "silu", b, "nhwc", path=rt.PATH_AUTO)
    assert np.array_equal(y_a, y_t)                      # auto picks the tensor path here
    assert orc.rel_err(y_t, y_f) <= 1e-2                 # same fp32 accumulation, different order: one bf16 ulp at most
    assert (y_t != y_f).mean() < 0.05
    _no_timeout()
    packed.close()


def test_tensor_path_channel_slice_and_batch_sampled():
    masks = _table(3)
    N, Cin, Cout, H, W = 8, 128, 128, 80, 80
    x = synth.round_like(synth.activations(23, 1, N, Cin, H, W), "bf16")
    w = synth.kaiming_weights(23, 1, Cout, Cin, 3)
    b = synth.bias(23, 1, Cout)
    _, packed = gu.select_pack(w, 3, masks, 3, "bf16")
    _, wd, _ = gu.oracle_weights(w, 3, masks, 3, "bf16")
    y = gu.run_conv(packed, 3, x, "bf16", 1, "silu", b, "nhwc", y_off=61, y_stride=251, path=rt.PATH_TENSOR)
    assert (y[:, :61] == 7.0).all() and (y[:, 189:] == 7.0).all()
    rng = np.random.default_rng(7)
    npts = 4000
    idx = np.stack([rng.integers(0, N, npts), rng.integers(0, Cout, npts), rng.integers(0, H, npts),
                    rng.integers(0, W, npts)], axis=1).astype(np.int32)
    idx[:4] = [[0, 0, 0, 0], [0, 0, 0, W - 1], [N - 1, Cout - 1, H - 1, W - 1], [N - 1, 0, H - 1, 0]]
    ref = orc.conv_points(3, x, wd, b, 1, orc.ACT_SILU, orc.DT_BF16, idx)
    got = y[idx[:, 0], 61 + idx[:, 1], idx[:, 2], idx[:, 3]]
    rms = float(np.sqrt(np.mean(ref.astype(np.float64) ** 2)))
    assert np.max(np.abs(got - ref) / np.maximum(np.abs(ref), rms)) <= 2e-2
    _no_timeout()
    packed.close()


def test_tensor_path_refuses_what_it_cannot_take():
    masks = _table(4)
    w = synth.kaiming_weights(24, 1, 64, 64, 3)
    _, packed = gu.select_pack(w, 3, masks, 4, "bf16")
    x = synth.round_like(synth.activations(24, 1, 1, 64, 8, 8), "bf16")
    with pytest.raises(rt.RtossError) as e:                                  # NCHW is not taken by the tensor path
        gu.run_conv(packed, 3, x, "bf16", 1, "none", None, "nchw", path=rt.PATH_TENSOR)
    assert e.value.status == 3
    y = gu.run_conv(packed, 3, x, "bf16", 1, "none", None, "nchw", path=rt.PATH_AUTO)   # auto falls back to FMA
    assert np.isfinite(y).all()
    packed.close()
    w8 = synth.kaiming_weights(24, 2, 16, 12, 3)                             # Cin not a multiple of 8
    _, packed = gu.select_pack(w8, 3, masks, 4, "bf16")
    x8 = synth.round_like(synth.activations(24, 2, 1, 12, 8, 8), "bf16")
    with pytest.raises(rt.RtossError) as e:
        gu.run_conv(packed, 3, x8, "bf16", 1, "none", None, "nhwc", path=rt.PATH_TENSOR)
    assert e.value.status == 3
    packed.close()


# Narrow layers run with the positions as the M operand of the MMA (filters as N): cases that differ there --
# filter counts around the 16-column read, one or two halves of 128 positions per tile, many tiles per CTA
NARROW = [
    # ksize, stride, N, Cin, Cout, H, W, k, dt, act, bias
    (1, 1, 1, 64, 8, 12, 10, 4, "bf16", "silu", True),       # one 16-filter read, half of it real; 120 positions: one half
    (1, 1, 1, 32, 64, 9, 16, 3, "f16", "none", False),       # 144 positions: two halves, the second nearly empty
    (1, 1, 4, 64, 32, 160, 160, 4, "bf16", "silu", True),    # several tiles per CTA, both accumulator stages in turn
    (3, 1, 2, 32, 32, 64, 64, 4, "bf16", "relu", True),      # half-filled channel block: two of four K slabs issued
    (3, 1, 1, 48, 40, 33, 21, 2, "f16", "silu", True),       # ragged filter count (40 of 48 columns), ragged channels
    (3, 2, 3, 16, 64, 31, 45, 3, "bf16", "silu", True),      # stride 2, odd sizes
    (1, 2, 2, 256, 48, 40, 40, 4, "bf16", "relu", False),    # deep K, strided 1x1
    (1, 1, 2, 32, 32, 40, 40, 4, "bf16", "silu", True),      # 32 channels: 64-byte rows, positions on M, many tiles
    (3, 2, 2, 32, 64, 64, 64, 4, "bf16", "silu", True),      # 32 channels, stride 2: four 64-byte-row sub-tiles per block
    (3, 1, 1, 24, 32, 20, 260, 3, "f16", "relu", True),      # 24 of 32 channels, column segments
]


@pytest.mark.parametrize("case", NARROW, ids=lambda c: "-".join(str(v) for v in c))
def test_tensor_path_narrow_layers(case):
    ks, s, N, Cin, Cout, H, W, k, dt, act, use_bias = case
    gu.check_layer(26, 900 + Cin + Cout + W, ks, N, Cin, Cout, H, W, s, k, _table(k), dt, act, "nhwc", use_bias=use_bias,
                   path=rt.PATH_TENSOR)
    _no_timeout()


@pytest.mark.parametrize("y_off,y_stride", [(8, 96), (5, 77)])
def test_tensor_path_narrow_channel_slice(y_off, y_stride):
    """Output written into a channel slice: aligned (16-byte stores) and unaligned (element stores); the rest of
    the buffer keeps its fill value."""
    masks = _table(4)
    N, Cin, Cout, H, W = 2, 64, 32, 19, 23
    x = synth.round_like(synth.activations(27, 1, N, Cin, H, W), "bf16")
    w = synth.kaiming_weights(27, 1, Cout, Cin, 3)
    b = synth.bias(27, 1, Cout)
    _, packed = gu.select_pack(w, 3, masks, 4, "bf16")
    _, wd, _ = gu.oracle_weights(w, 3, masks, 4, "bf16")
    y = gu.run_conv(packed, 3, x, "bf16", 1, "silu", b, "nhwc", y_off=y_off, y_stride=y_stride, path=rt.PATH_TENSOR)
    assert (y[:, :y_off] == 7.0).all() and (y[:, y_off + Cout:] == 7.0).all()
    ref = gu.oracle_conv(3, x, wd, b, 1, "silu", "bf16")
    assert orc.rel_err(y[:, y_off:y_off + Cout], ref) <= gu.TOL["bf16"]
    _no_timeout()
    packed.close()


MANY_TILES = [
    # ks, stride, N, Cin, Cout, H, W, k, dtype, act: several tiles per CTA, so the operand rings wrap and their phase
    # parities flip inside one CTA while the MMA thread's early look at the next stages crosses tile boundaries
    (1, 1, 2, 320, 192, 120, 136, 4, "bf16", "silu"),    # five channel blocks per tile, ragged last block, two filter tiles
    (1, 1, 2, 136, 48, 150, 200, 3, "bf16", "relu"),     # positions on M, three channel blocks (the last one 8 channels)
    (3, 1, 2, 64, 64, 200, 272, 4, "bf16", "silu"),      # 3x3, one channel block per tile, about three tiles per CTA
    (3, 2, 2, 128, 128, 160, 200, 4, "f16", "none"),     # stride 2: four staged sub-tiles per activation stage
]


@pytest.mark.parametrize("case", MANY_TILES, ids=lambda c: "-".join(str(v) for v in c))
def test_tensor_path_many_tiles_per_cta(case):
    ks, s, N, Cin, Cout, H, W, k, dt, act = case
    gu.check_layer(27, 900 + Cin + W, ks, N, Cin, Cout, H, W, s, k, _table(k), dt, act, "nhwc", path=rt.PATH_TENSOR)
    _no_timeout()
