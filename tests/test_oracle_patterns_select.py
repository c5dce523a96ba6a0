"""Pins for the CPU oracle: pattern tables (Section IV.B, Eq. 1, criterion 1),
selection (Algorithm 2) and the 1x1 regrouping (Algorithm 3).  None of the
expectations below is produced by the oracle itself."""
import itertools
import math
import os
from fractions import Fraction

import numpy as np
import pytest

from oracle import rtoss_oracle as orc
from paper_2303_02191_b200 import synth

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def _golden_tables():
    out = {}
    for line in open(os.path.join(GOLD, "pattern_tables.txt")):
        if line.startswith("#") or not line.strip():
            continue
        name, *vals = line.split()
        out[name] = [int(v, 16) for v in vals]
    return out


def _taps(m):
    return [t for t in range(9) if (m >> t) & 1]


def _connected_py(m):
    taps = set(_taps(m))
    start = min(taps)
    seen, todo = {start}, [start]
    while todo:
        t = todo.pop()
        r, c = divmod(t, 3)
        for rr, cc in ((r - 1, c), (r + 1, c), (r, c - 1), (r, c + 1)):
            u = 3 * rr + cc
            if 0 <= rr < 3 and 0 <= cc < 3 and u in taps and u not in seen:
                seen.add(u)
                todo.append(u)
    return seen == taps


# ---------------------------------------------------------------- tables

@pytest.mark.parametrize("k", range(1, 10))
def test_all_preset_has_binomial_count(k):
    masks = orc.pattern_preset(k, orc.PRESET_ALL)
    assert len(masks) == math.comb(9, k)          # Eq. (1)
    assert len(set(masks.tolist())) == len(masks)
    assert all(bin(int(m)).count("1") == k for m in masks)
    assert list(masks) == sorted(masks)


def test_eq1_counts_quoted_values():
    assert [len(orc.pattern_preset(k, orc.PRESET_ALL)) for k in (2, 3, 4, 5)] == [36, 84, 126, 126]


def test_conn4_counts_closed_form():
    # k=2: edges of the 3x3 grid graph = 2*3*2; k=3: two-edge paths =
    # sum over vertices of C(deg,2) = 4*1 + 4*3 + 6 (the grid has no triangles).
    assert len(orc.pattern_preset(2, orc.PRESET_CONN4)) == 12
    assert len(orc.pattern_preset(3, orc.PRESET_CONN4)) == 4 * 1 + 4 * 3 + 6


@pytest.mark.parametrize("k,count", [(1, 9), (2, 12), (3, 22), (4, 36), (5, 49), (9, 1)])
def test_conn4_against_python_flood_fill(k, count):
    want = [m for m in range(1, 512) if bin(m).count("1") == k and _connected_py(m)]
    got = orc.pattern_preset(k, orc.PRESET_CONN4).tolist()
    assert got == want
    assert len(got) == count


def test_golden_tables():
    g = _golden_tables()
    assert orc.pattern_preset(2, orc.PRESET_CONN4).tolist() == g["CONN4_2"]
    assert orc.pattern_preset(3, orc.PRESET_CONN4).tolist() == g["CONN4_3"]
    assert orc.pattern_preset(4, orc.PRESET_CENTRE8).tolist() == g["CENTRE8"]
    assert orc.pattern_preset(9, orc.PRESET_DENSE).tolist() == [0x1FF]


def _d4_images(m):
    def apply(f):
        return sum(1 << f(*divmod(t, 3)) for t in _taps(m))
    rot = lambda r, c: 3 * c + (2 - r)
    flip = lambda r, c: 3 * r + (2 - c)
    out, cur = [], m
    for _ in range(4):
        cur = sum(1 << rot(*divmod(t, 3)) for t in _taps(cur))
        out.append(cur)
        out.append(sum(1 << flip(*divmod(t, 3)) for t in _taps(cur)))
    return out


@pytest.mark.parametrize("k,preset", [(2, 1), (3, 1), (4, 1), (5, 1), (4, 2), (3, 0)])
def test_presets_closed_under_square_symmetries(k, preset):
    masks = set(orc.pattern_preset(k, preset).tolist())
    for m in masks:
        assert set(_d4_images(m)) <= masks


def test_centre8_properties():
    masks = orc.pattern_preset(4, orc.PRESET_CENTRE8).tolist()
    assert len(masks) == 8
    for m in masks:
        assert (m >> 4) & 1 and _connected_py(m) and bin(m).count("1") == 4
    conn_centre = [m for m in orc.pattern_preset(4, orc.PRESET_CONN4).tolist() if (m >> 4) & 1]
    assert len(conn_centre) == 28 and set(masks) <= set(conn_centre)


def test_table_validation():
    assert orc.pattern_table_valid([0x01B, 0x036], 4)
    assert not orc.pattern_table_valid([0x01B, 0x01B], 4)      # duplicate
    assert not orc.pattern_table_valid([0x01B, 0x007], 4)      # popcount
    assert not orc.pattern_table_valid([0x200 | 0x7], 4)       # outside the 9 taps
    assert not orc.pattern_table_valid([0], 1)
    with pytest.raises(ValueError):
        orc.pattern_preset(3, orc.PRESET_CENTRE8)
    with pytest.raises(ValueError):
        orc.pattern_preset(4, orc.PRESET_DENSE)


# ---------------------------------------------------------------- select

def _exact_sums(kernel, masks):
    return [sum(Fraction(float(kernel[t])) ** 2 for t in _taps(m)) for m in masks]


def test_worked_example_from_golden_file():
    rows = {}
    for line in open(os.path.join(GOLD, "select_worked_example.txt")):
        if line.startswith("#") or not line.strip():
            continue
        key, *vals = line.split()
        rows[key] = [float(v) for v in vals]
    masks = _golden_tables()["CENTRE8"]
    kern = np.array(rows["kernel"], dtype=np.float32)
    pid = orc.select_kernels(kern, masks)
    assert int(pid[0]) == int(rows["pid"][0])
    wm = orc.mask_3x3(kern.reshape(1, 1, 3, 3), masks, pid.reshape(1, 1))
    assert [v for v in wm.ravel().tolist() if v != 0.0] == rows["kept"]
    val, perm, off = orc.pack_3x3(kern.reshape(1, 1, 3, 3), masks, 4, pid.reshape(1, 1), orc.DT_F32)
    assert val.tolist() == rows["kept"]


@pytest.mark.parametrize("k", [1, 2, 3, 4, 5, 8])
def test_select_is_first_exact_argmax_over_all_subsets(k):
    masks = orc.pattern_preset(k, orc.PRESET_ALL).tolist()
    w = synth.normal(11, k, (300, 9))
    pid = orc.select_kernels(w, masks)
    near_ties = 0
    for i in range(w.shape[0]):
        s = _exact_sums(w[i], masks)
        best = max(s)
        if s[pid[i]] != best or s.index(best) != pid[i]:
            # only allowed when float rounding could reorder: sums within 2^-20 relative
            assert abs(s[pid[i]] - best) <= best * Fraction(1, 2 ** 20)
            near_ties += 1
    assert near_ties <= 3


@pytest.mark.parametrize("k", [2, 3, 4])
def test_all_table_keeps_the_k_largest_magnitudes(k):
    masks = orc.pattern_preset(k, orc.PRESET_ALL)
    w = synth.normal(5, 100 + k, (500, 9))
    pid = orc.select_kernels(w, masks)
    for i in range(w.shape[0]):
        order = np.argsort(-np.abs(w[i].astype(np.float64)), kind="stable")
        gap = abs(w[i][order[k - 1]]) - abs(w[i][order[k]])
        if gap < 1e-4:
            continue
        assert sorted(order[:k].tolist()) == _taps(int(masks[pid[i]]))


def test_single_pattern_table_gives_zero():
    w = synth.normal(1, 1, (64, 9))
    assert not orc.select_kernels(w, [0x01B]).any()


def test_invariance_to_power_of_two_scale_and_sign_flips():
    masks = orc.pattern_preset(3, orc.PRESET_CONN4)
    w = synth.normal(2, 3, (400, 9))
    pid = orc.select_kernels(w, masks)
    assert np.array_equal(pid, orc.select_kernels(w * np.float32(0.125), masks))
    assert np.array_equal(pid, orc.select_kernels(w * np.float32(1024.0), masks))
    signs = np.where(synth.normal(2, 4, (400, 9)) > 0, 1.0, -1.0).astype(np.float32)
    assert np.array_equal(pid, orc.select_kernels(w * signs, masks))


def test_equivariance_under_a_rotation_of_the_taps():
    masks = orc.pattern_preset(4, orc.PRESET_CENTRE8).tolist()
    w = synth.normal(3, 5, (300, 9))
    rot = [3 * c + (2 - r) for r in range(3) for c in range(3)]   # tap t moves to rot[t]
    wr = np.zeros_like(w)
    wr[:, rot] = w
    rmask = lambda m: sum(1 << rot[t] for t in _taps(m))
    pid, pidr = orc.select_kernels(w, masks), orc.select_kernels(wr, masks)
    checked = 0
    for i in range(w.shape[0]):
        s = sorted(_exact_sums(w[i], masks), reverse=True)
        if s[0] - s[1] < Fraction(1, 10 ** 4):
            continue
        assert masks[pidr[i]] == rmask(masks[pid[i]])
        checked += 1
    assert checked > 200


def test_ties_go_to_the_lowest_pattern_and_nan_never_wins():
    masks = [0x003, 0x006, 0x180]
    ones = np.ones(9, dtype=np.float32)
    assert orc.select_kernels(ones, masks)[0] == 0
    kern = np.zeros(9, dtype=np.float32)
    kern[7] = kern[8] = 2.0
    assert orc.select_kernels(kern, masks)[0] == 2
    kern[0] = np.nan                      # pattern 0 has a NaN sum; pattern 1 (taps 1,2) is 0, pattern 2 is 8
    assert orc.select_kernels(kern, masks)[0] == 2
    allnan = np.full(9, np.nan, dtype=np.float32)
    assert orc.select_kernels(allnan, masks)[0] == 0
    kern = np.zeros(9, dtype=np.float32)
    assert orc.select_kernels(kern, masks)[0] == 0


def test_select_uses_float32_rounding_of_squares_and_sums():
    # 1 + 2^-24 + 2^-24: float32 adds left to right give 1 (each half-ulp tie rounds to even),
    # while exact arithmetic gives 1 + 2^-23 > 1.  Pattern 1 = {tap 3} holds exactly 1+2^-23.
    e = np.float32(2.0 ** -12)            # e*e = 2^-24
    kern = np.zeros(9, dtype=np.float32)
    kern[0], kern[1], kern[2] = 1.0, e, e
    kern[3] = np.sqrt(np.float64(1 + 2.0 ** -23)).astype(np.float32)
    masks = [0x007, 0x008 | 0x010 | 0x020]
    q3 = np.float32(kern[3]) * np.float32(kern[3])
    expect = 1 if q3 > np.float32(1.0) else 0
    assert orc.select_kernels(kern, masks)[0] == expect


# ---------------------------------------------------------------- 1x1 (Algorithm 3)

@pytest.mark.parametrize("cout,cin", [(128, 256), (7, 5), (16, 9), (3, 3), (2, 4), (1, 8)])
def test_1x1_select_equals_3x3_select_on_reshaped_runs(cout, cin):
    masks = orc.pattern_preset(3, orc.PRESET_CONN4)
    w = synth.kaiming_weights(0, 77, cout, cin, 1).reshape(cout, cin)
    pid1 = orc.select_1x1(w, masks)
    G = (cout * cin) // 9
    assert len(pid1) == G
    if G:
        ref = orc.select_kernels(w.ravel()[:9 * G].reshape(G, 9), masks)
        assert np.array_equal(pid1, ref)
    wm = orc.mask_1x1(w, masks, pid1).ravel()
    assert not wm[9 * G:].any()                       # left-over weights are pruned
    assert all(np.count_nonzero(wm[9 * g:9 * g + 9]) == 3 for g in range(G))


def test_1x1_group_count_of_the_256_to_128_layer():
    w = synth.kaiming_weights(0, 78, 128, 256, 1).reshape(128, 256)
    pid1 = orc.select_1x1(w, orc.pattern_preset(2, orc.PRESET_CONN4))
    assert len(pid1) == 3640 and 128 * 256 - 9 * 3640 == 8


def test_1x1_flat_order_is_filter_major():
    # weights 0..17 laid out [Cout=2][Cin=9]: run 0 must be filter 0's nine weights
    w = np.zeros((2, 9), dtype=np.float32)
    w[0, :2] = 5.0          # taps 0,1 of run 0
    w[1, 7:] = 5.0          # taps 7,8 of run 1
    masks = orc.pattern_preset(2, orc.PRESET_CONN4).tolist()
    pid1 = orc.select_1x1(w, masks)
    assert masks[pid1[0]] == 0x003 and masks[pid1[1]] == 0x180


# ---------------------------------------------------------------- criterion 2: usage ranking and the cut

def test_usage_of_one_tap_and_eight_tap_patterns_is_uniform():
    """Closed form: for nine i.i.d. values every tap is equally likely to be the largest (1-entry patterns keep it)
    and equally likely to be the smallest (8-entry patterns drop it): each of the nine patterns wins 1/9 of the
    sample, within five standard deviations of the binomial count."""
    n = 90000
    sample = synth.uniform_kernels(11, n)
    sd = math.sqrt(n * (1 / 9) * (8 / 9))
    for k in (1, 8):
        masks = orc.pattern_preset(k, orc.PRESET_ALL)
        counts = orc.pattern_usage(sample, masks)
        assert int(counts.sum()) == n and len(counts) == 9
        assert np.all(np.abs(counts.astype(float) - n / 9) < 5 * sd)


def test_usage_counts_against_a_pure_python_argmax():
    masks = orc.pattern_preset(3, orc.PRESET_CONN4)
    sample = synth.uniform_kernels(12, 500)
    want = np.zeros(len(masks), dtype=np.uint64)
    for kern in sample.reshape(-1, 9):
        sq = [float(np.float32(v) * np.float32(v)) for v in kern]
        best, best_e = 0, -1.0
        for p, m in enumerate(masks):
            e = np.float32(0)
            for t in range(9):
                if (int(m) >> t) & 1:
                    e = np.float32(e + np.float32(sq[t]))
            if float(e) > best_e:
                best, best_e = p, float(e)
        want[best] += 1
    assert np.array_equal(orc.pattern_usage(sample, masks), want)


def test_usage_is_symmetric_under_the_squares_symmetries():
    """A uniform sample has no preferred direction: patterns that are rotations / reflections of one another (one
    orbit of the square's symmetry group) are used equally often up to sampling noise.  The twelve dominoes fall into
    two orbits: eight touching a corner, four touching the centre."""
    def image(mask, f):
        out = 0
        for t in range(9):
            if (mask >> t) & 1:
                r, c = divmod(t, 3)
                r2, c2 = f(r, c)
                out |= 1 << (3 * r2 + c2)
        return out
    syms = [lambda r, c: (r, c), lambda r, c: (c, 2 - r), lambda r, c: (2 - r, 2 - c), lambda r, c: (2 - c, r),
            lambda r, c: (r, 2 - c), lambda r, c: (2 - r, c), lambda r, c: (c, r), lambda r, c: (2 - c, 2 - r)]
    masks = [int(m) for m in orc.pattern_preset(2, orc.PRESET_CONN4)]
    counts = orc.pattern_usage(synth.uniform_kernels(13, 120000), masks).astype(float)
    orbits = {}
    for m, c in zip(masks, counts):
        orbits.setdefault(min(image(m, f) for f in syms), []).append(c)
    assert sorted(len(v) for v in orbits.values()) == [4, 8]
    for v in orbits.values():
        assert max(v) / min(v) < 1.1


def test_rank_orders_by_count_then_mask_and_returns_a_table():
    masks = np.array([0x003, 0x006, 0x009, 0x012, 0x018, 0x024], dtype=np.uint16)
    counts = np.array([5, 9, 5, 0, 9, 7], dtype=np.uint64)
    top, order = orc.pattern_rank(masks, counts, 4)
    assert list(order) == [1, 4, 5, 0, 2, 3]                 # 9 (mask 0x006), 9 (0x018), 7, 5 (0x003), 5 (0x009), 0
    assert list(top) == [0x003, 0x006, 0x018, 0x024]         # the four best, ascending
    assert orc.pattern_table_valid(top, 2)
    full, _ = orc.pattern_rank(masks, counts, 6)
    assert np.array_equal(full, masks)                       # keeping all candidates returns the table itself
    one, _ = orc.pattern_rank(masks, counts, 1)
    assert list(one) == [0x006]                              # the tie at 9 goes to the lower mask


def test_derive_keeps_a_subset_with_the_largest_counts():
    sample = synth.uniform_kernels(14, 40000)
    top, cand, counts = orc.derive_pattern_table(sample, 3, orc.PRESET_CONN4, 8)
    assert len(top) == 8 and set(top) <= set(cand) and orc.pattern_table_valid(top, 3)
    kept = np.isin(cand, top)
    assert counts[kept].min() >= counts[~kept].max()
    everything, _, _ = orc.derive_pattern_table(sample, 3, orc.PRESET_CONN4, 1000)
    assert np.array_equal(everything, cand)
    # Eq. 1 alone as the candidate family: the most used 4-entry patterns over all 126
    top4, cand4, _ = orc.derive_pattern_table(sample, 4, orc.PRESET_ALL, 21)
    assert len(cand4) == math.comb(9, 4) and len(top4) == 21
