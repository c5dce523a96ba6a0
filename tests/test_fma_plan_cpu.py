"""Host arithmetic of the FMA path's staging plan (rtoss_fma_plan3x3): every activation vector the kernel would
fetch through cp.async starts on a multiple of its size.  The finer kernel shape (four pixels per lane) once faulted with
a misaligned address on a 64-channel 40 x 40 bf16 NCHW layer: with an odd number of lane columns every second tile
started 8 bytes off a 16-byte boundary while the vector width had been chosen from the row pitch alone.  Checked tile
by tile and vector by vector over shapes that exercise both kernel shapes, all three types and both strides."""
import itertools

import pytest

from paper_2303_02191_b200 import binding as rt

ES = {rt.F32: 4, rt.BF16: 2, rt.F16: 2}


def _check(N, H, W, stride, dt, Cin, Cout, k=4):
    p = rt.rtoss_fma_plan3x3(N, H, W, stride, rt.NCHW, dt, Cin, Cout, k)
    assert not p.small_cin
    es = ES[dt]
    Ho, Wo = (H - 1) // stride + 1, (W - 1) // stride + 1
    assert p.tiles_x * p.lanes_x * p.pixels_per_lane >= Wo and p.tiles_y * p.lanes_y >= Ho
    assert p.lanes_x * p.lanes_y <= 32
    assert p.grid_x == p.tiles_x * p.tiles_y * N
    assert p.shared_bytes <= 227 * 1024 // p.ctas_per_sm
    if p.staging != 1:
        return p
    vb = p.vector_bytes
    assert vb in (4, 8, 16) and vb >= es
    veq = vb // es
    nv = p.vectors_per_plane // p.staged_rows
    assert nv * p.staged_rows == p.vectors_per_plane
    assert (W * es) % vb == 0                       # row pitch, hence every plane and image offset
    for tx in range(p.tiles_x):
        ox0 = tx * p.lanes_x * p.pixels_per_lane
        for j in range(nv):
            ix = ox0 * stride - veq + j * veq      # first element of vector j of a staged row
            assert (ix * es) % vb == 0, (tx, j, ix)
    # the vectors of a staged row cover its columns ox0*S - 1 .. ox0*S - 1 + staged_cols - 1
    assert nv * veq >= p.staged_cols + veq - 1
    return p


def test_the_layer_that_faulted_takes_the_finer_shape_with_a_narrower_vector():
    p = _check(1, 40, 40, 1, rt.BF16, 64, 64)
    assert p.pixels_per_lane == 4 and p.grid_x * p.grid_y >= 16
    # (five lane columns of four pixels: tiles 20 pixels = 40 bytes apart, so 8-byte vectors)
    if p.lanes_x % 2:
        assert p.vector_bytes <= 8


def test_small_fp32_layer_spreads_over_many_ctas():
    p = _check(1, 32, 32, 1, rt.F32, 32, 32)
    assert p.pixels_per_lane == 4
    assert p.grid_x * p.grid_y >= 16       # four CTAs with the coarse shape


SHAPES = [(1, 40, 40), (1, 20, 20), (2, 13, 16), (1, 7, 12), (8, 80, 80), (1, 25, 36), (1, 160, 160), (3, 10, 200), (1, 9, 8)]


@pytest.mark.parametrize("shape,dt,stride,ch", list(itertools.product(SHAPES, (rt.F32, rt.BF16, rt.F16), (1, 2),
                                                                         ((64, 64), (32, 48), (128, 16), (8, 200)))))
def test_every_vector_address_is_aligned(shape, dt, stride, ch):
    N, H, W = shape
    _check(N, H, W, stride, dt, ch[0], ch[1])


def test_argument_errors_and_small_cin():
    with pytest.raises(rt.RtossError):
        rt.rtoss_fma_plan3x3(1, 8, 8, 3, rt.NCHW, rt.F32, 16, 16, 4)
    assert rt.rtoss_fma_plan3x3(1, 64, 64, 2, rt.NHWC, rt.BF16, 3, 32, 4).small_cin == 1
