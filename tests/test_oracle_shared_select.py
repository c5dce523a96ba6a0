"""Pins of the oracle's block-shared pattern selection (`oracle_select_shared`: one pattern per block of FB filters x
CB input channels, the pattern that retains the most energy of the block; a variant of Section IV.C's shared kernel
masks).  None of these uses the function to make its own expectation: a hand-worked example, exact rational
arithmetic over every pattern, the reduction to Algorithm 2 for blocks of one kernel, and structural properties."""
import os
from fractions import Fraction

import numpy as np
import pytest

from oracle import rtoss_oracle as orc
from paper_2303_02191_b200 import synth

GOLDEN = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden")


def _exact_block_argmax(w, masks, FB, CB):
    """Exact rational arithmetic on the float32 squares: per block the first pattern with the largest sum, plus
    whether the runner-up is so close that float rounding of the sums could matter (relative gap below 1e-12)."""
    Cout, Cin = w.shape[:2]
    q = (w.astype(np.float32) * w.astype(np.float32)).astype(np.float32).reshape(Cout, Cin, 9)
    pid = np.zeros((Cout, Cin), dtype=np.uint8)
    close = np.zeros((Cout, Cin), dtype=bool)
    for co0 in range(0, Cout, FB):
        for ci0 in range(0, Cin, CB):
            blk = q[co0:co0 + FB, ci0:ci0 + CB].reshape(-1, 9)
            E = [sum(Fraction(float(v)) for v in blk[:, t]) for t in range(9)]
            S = [sum(E[t] for t in range(9) if (int(m) >> t) & 1) for m in masks]
            best = max(range(len(S)), key=lambda p: (S[p], -p))
            pid[co0:co0 + FB, ci0:ci0 + CB] = best
            others = [S[p] for p in range(len(S)) if p != best]
            if others and S[best] > 0 and (S[best] - max(others)) / S[best] < Fraction(1, 10 ** 12):
                close[co0:co0 + FB, ci0:ci0 + CB] = True
    return pid, close


def test_hand_worked_block_example():
    vals = {}
    for line in open(os.path.join(GOLDEN, "select_shared_worked_example.txt")):
        if line.startswith("#") or not line.strip():
            continue
        key, rest = line.split(None, 1)
        vals[key] = rest.split()
    masks = np.array([int(v, 16) for v in vals["masks"]], dtype=np.uint16)
    w = np.array([[float(v) for v in vals["kernelA"]], [float(v) for v in vals["kernelB"]]], dtype=np.float32).reshape(2, 1, 3, 3)
    assert orc.select_3x3(w, masks).ravel().tolist() == [int(v) for v in vals["per_kernel_pid"]]
    assert orc.select_shared(w, masks, 2, 1).ravel().tolist() == [int(v) for v in vals["shared_pid"]]
    # the same two kernels side by side as channels of one filter: a block of 1 x 2
    w2 = w.reshape(1, 2, 3, 3)
    assert orc.select_shared(w2, masks, 1, 2).ravel().tolist() == [int(v) for v in vals["shared_pid"]]


@pytest.mark.parametrize("FB,CB,k", [(1, 1, 4), (2, 3, 4), (4, 4, 3), (8, 16, 2), (5, 7, 4), (128, 16, 4)])
def test_first_exact_argmax_of_the_block_energy(FB, CB, k):
    """Brute force with exact rational sums on small layers, ragged blocks included (Cout, Cin no multiples)."""
    preset = orc.PRESET_CENTRE8 if k == 4 else orc.PRESET_CONN4
    masks = orc.pattern_preset(k, preset)
    Cout, Cin = (11, 10) if FB < 128 else (130, 20)
    w = synth.kaiming_weights(61, FB * 100 + CB, Cout, Cin, 3)
    want, close = _exact_block_argmax(w, masks, FB, CB)
    got = orc.select_shared(w, masks, FB, CB)
    assert not close.all()
    assert np.array_equal(got[~close], want[~close])
    assert close.sum() <= 0.01 * close.size


def test_blocks_of_one_kernel_are_algorithm_2():
    """FB = CB = 1: the block is one kernel; the choice is Algorithm 2's (float there, double here: kernels whose two
    best sums agree to 1e-6 are left out of the comparison)."""
    masks = orc.pattern_preset(3, orc.PRESET_CONN4)
    w = synth.kaiming_weights(62, 1, 24, 20, 3)
    a = orc.select_3x3(w, masks)
    b = orc.select_shared(w, masks, 1, 1)
    q = (w.astype(np.float64) ** 2).reshape(24, 20, 9)
    S = np.stack([q[..., [t for t in range(9) if (int(m) >> t) & 1]].sum(-1) for m in masks], -1)
    top2 = np.sort(S, -1)[..., -2:]
    clear = (top2[..., 1] - top2[..., 0]) > 1e-6 * top2[..., 1]
    assert clear.mean() > 0.99
    assert np.array_equal(a[clear], b[clear])


def test_ids_are_constant_inside_blocks_and_keep_exactly_k_taps():
    masks = orc.pattern_preset(4, orc.PRESET_CENTRE8)
    Cout, Cin, FB, CB = 40, 36, 16, 8
    w = synth.kaiming_weights(63, 1, Cout, Cin, 3)
    pid = orc.select_shared(w, masks, FB, CB)
    for co0 in range(0, Cout, FB):
        for ci0 in range(0, Cin, CB):
            assert len(np.unique(pid[co0:co0 + FB, ci0:ci0 + CB])) == 1
    wm = orc.mask_3x3(w, masks, pid)
    kept = (wm.reshape(Cout, Cin, 9) != 0).sum(-1)
    assert (kept == 4).all()                      # every kernel keeps its k taps, none is removed
    assert abs(w.size / np.count_nonzero(wm) - 9 / 4) < 1e-12    # the compression of the per-kernel method, 9 / k
    # the block's retained energy is what was maximised: no other pattern keeps more of it
    q = (w.astype(np.float64) ** 2).reshape(Cout, Cin, 9)
    for co0 in range(0, Cout, FB):
        for ci0 in range(0, Cin, CB):
            E = q[co0:co0 + FB, ci0:ci0 + CB].reshape(-1, 9).sum(0)
            S = [sum(E[t] for t in range(9) if (int(m) >> t) & 1) for m in masks]
            assert S[int(pid[co0, ci0])] >= max(S) * (1 - 1e-12)


def test_a_block_of_identical_kernels_and_scale_invariance():
    masks = orc.pattern_preset(4, orc.PRESET_CENTRE8)
    one = synth.kaiming_weights(64, 1, 1, 1, 3)
    w = np.tile(one, (8, 4, 1, 1))
    assert (orc.select_shared(w, masks, 8, 4) == orc.select_3x3(one, masks)[0, 0]).all()
    w = synth.kaiming_weights(64, 2, 16, 16, 3)
    a = orc.select_shared(w, masks, 8, 8)
    assert np.array_equal(a, orc.select_shared(w * np.float32(-4.0), masks, 8, 8))   # power-of-two scale and sign: exact


def test_shared_selection_retains_less_than_per_kernel_selection_but_never_more():
    """Sharing a pattern can only lose retained energy against the free per-kernel choice (which is optimal kernel by
    kernel), and a single pattern table makes both the same."""
    masks = orc.pattern_preset(4, orc.PRESET_CENTRE8)
    w = synth.kaiming_weights(65, 1, 32, 32, 3)
    free = orc.mask_3x3(w, masks, orc.select_3x3(w, masks))
    shared = orc.mask_3x3(w, masks, orc.select_shared(w, masks, 16, 16))
    e_free, e_shared = float((free.astype(np.float64) ** 2).sum()), float((shared.astype(np.float64) ** 2).sum())
    assert e_shared < e_free
    assert e_shared > 0.4 * float((w.astype(np.float64) ** 2).sum())   # four taps of nine keep at least 4/9 on i.i.d. weights
    one = masks[:1]
    assert np.array_equal(orc.select_shared(w, one, 16, 16), orc.select_3x3(w, one))
