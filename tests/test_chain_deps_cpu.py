"""Host logic of rtoss_conv_chain: which earlier convolutions a convolution has to wait for, derived from the byte
ranges of the operands (no GPU: plain arithmetic through the C ABI), against a brute-force check byte by byte."""
import itertools
import random

import pytest

from paper_2303_02191_b200 import binding as rt


def brute(spans):
    """bit j of out[i]: i reads a byte j writes, or writes a byte j reads or writes."""
    def bytes_of(lo, hi):
        return set(range(lo, hi))
    out = []
    for i, (xl, xh, yl, yh, rl, rh) in enumerate(spans):
        m = 0
        for j in range(i):
            jx, jy, jr = bytes_of(*spans[j][0:2]), bytes_of(*spans[j][2:4]), bytes_of(*spans[j][4:6])
            reads = (bytes_of(xl, xh) | bytes_of(rl, rh)) & jy
            writes = bytes_of(yl, yh) & (jx | jy | jr)
            if reads or writes:
                m |= 1 << j
        out.append(m)
    return out


def test_bottleneck_block_by_hand():
    # in = [0,100), t1 = [100,200), t2 = [200,300), idn = [300,400), out = [400,500)
    spans = [
        (0, 100, 100, 200, 0, 0),        # conv1: in -> t1
        (0, 100, 300, 400, 0, 0),        # projection: in -> idn
        (100, 200, 200, 300, 0, 0),      # conv2: t1 -> t2
        (200, 300, 400, 500, 300, 400),  # conv3: t2 -> out, + idn
        (400, 500, 100, 200, 0, 0),      # next conv1 writes over t1: behind conv3 (its input), conv1 (same buffer) and conv2 (reads t1)
    ]
    assert rt.rtoss_chain_deps_spans(spans) == [0, 0, 0b001, 0b110, 0b1101]


def test_against_byte_by_byte_enumeration():
    rnd = random.Random(5)
    for _ in range(200):
        n = rnd.randint(1, 7)
        spans = []
        for _i in range(n):
            def span(may_be_empty=False):
                if may_be_empty and rnd.random() < 0.5:
                    return (0, 0)
                lo = rnd.randint(0, 40)
                return (lo, lo + rnd.randint(1, 12))
            spans.append(span() + span() + span(True))
        assert rt.rtoss_chain_deps_spans(spans) == brute(spans), spans


def test_touching_ranges_do_not_overlap_and_bad_arguments_are_refused():
    assert rt.rtoss_chain_deps_spans([(0, 8, 8, 16, 0, 0), (16, 24, 24, 32, 0, 0)]) == [0, 0]
    assert rt.rtoss_chain_deps_spans([(0, 8, 8, 16, 0, 0), (15, 24, 24, 32, 0, 0)]) == [0, 1]
    with pytest.raises(rt.RtossError):
        rt.rtoss_chain_deps_spans([(8, 0, 8, 16, 0, 0)])          # a range that ends before it starts
    with pytest.raises(rt.RtossError):
        rt.rtoss_chain_deps_spans([(0, 1, 1, 2, 0, 0)] * 33)       # more than 32 items
