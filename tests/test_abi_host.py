"""CPU-side checks of the C-ABI library: it loads, exports every function the
header declares, and its host-only entry points (pattern presets, table
validation, layer grouping) agree with the oracle.  No GPU compute here."""
import ctypes
import os
import re

import numpy as np
import pytest

from oracle import rtoss_oracle as orc
from paper_2303_02191_b200 import synth

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def rt():
    from paper_2303_02191_b200 import _build
    _build.build()
    from paper_2303_02191_b200 import binding
    return binding


def test_library_exports_every_declared_symbol(rt):
    header = open(os.path.join(ROOT, "include", "rtoss.h")).read()
    header = re.sub(r"/\*.*?\*/", "", header, flags=re.S)
    declared = set(re.findall(r"\b(rtoss_[a-z0-9_]+)\s*\(", header))
    assert declared == set(rt.SYMBOLS)
    raw = ctypes.CDLL(rt.LIB_PATH)
    for name in declared:
        assert hasattr(raw, name), name


def test_status_strings(rt):
    assert rt.status_string(0) == "ok"
    assert len({rt.status_string(s) for s in range(8)}) == 8


@pytest.mark.parametrize("k,preset", [(k, p) for k in range(1, 10) for p in (0, 1)] + [(4, 2), (9, 3)])
def test_presets_match_oracle(rt, k, preset):
    assert rt.rtoss_pattern_preset(k, preset).tolist() == orc.pattern_preset(k, preset).tolist()


def test_preset_errors(rt):
    with pytest.raises(rt.RtossError):
        rt.rtoss_pattern_preset(3, rt.PRESET_CENTRE8)
    with pytest.raises(rt.RtossError):
        rt.rtoss_pattern_preset(8, rt.PRESET_DENSE)
    with pytest.raises(rt.RtossError):
        rt.rtoss_pattern_preset(0, rt.PRESET_ALL)
    out = np.zeros(4, dtype=np.uint16)
    n = ctypes.c_int(4)                      # capacity too small for the 12 masks
    assert rt.lib.rtoss_pattern_preset(2, rt.PRESET_CONN4, out.ctypes.data_as(ctypes.c_void_p), ctypes.byref(n)) == 1


def test_table_validation_matches_oracle(rt):
    cases = [([0x01B, 0x036], 4), ([0x01B, 0x01B], 4), ([0x01B, 0x007], 4), ([0x207], 4), ([0], 1),
             (list(orc.pattern_preset(3, 1)), 3), ([0x1FF], 9), ([0x1FF], 8)]
    for masks, k in cases:
        assert (rt.rtoss_pattern_table_validate(masks, k) == 0) == orc.pattern_table_valid(masks, k)
    too_many = list(range(1, 257))
    assert rt.rtoss_pattern_table_validate(too_many, 1) == 2


def _random_dag(seed, L):
    rng = np.random.default_rng(seed)
    nodes = []
    for i in range(L):
        n_in = 0 if i == 0 else int(rng.integers(0, min(i, 3) + 1))
        inputs = [int(v) for v in rng.choice(i, size=n_in, replace=False)] if n_in else []
        if rng.random() < 0.6:
            c = int(rng.choice([8, 16]))
            nodes.append(dict(kind="conv", cin=c, cout=int(rng.choice([8, 16])), ksize=int(rng.choice([1, 3])), inputs=inputs))
        else:
            nodes.append(dict(kind="op", inputs=inputs))
    return nodes


@pytest.mark.parametrize("seed", range(6))
def test_group_layers_matches_oracle_on_random_dags(rt, seed):
    nodes = _random_dag(seed, 40)
    p0, g0, n0 = orc.group_layers(nodes)
    p1, g1, n1 = rt.rtoss_group_layers(nodes)
    assert p0.tolist() == p1.tolist() and g0.tolist() == g1.tolist() and n0 == n1


def test_group_layers_yolov5s_graph_and_errors(rt):
    nodes = synth.yolov5s_graph()
    p0, g0, n0 = orc.group_layers(nodes)
    p1, g1, n1 = rt.rtoss_group_layers(nodes)
    assert p0.tolist() == p1.tolist() and g0.tolist() == g1.tolist() and n0 == n1
    bad = [dict(kind="conv", cin=8, cout=8, ksize=3, inputs=[0])]       # input id not below the node's own
    with pytest.raises(rt.RtossError):
        rt.rtoss_group_layers(bad)
    bad = [dict(kind="conv", cin=8, cout=8, ksize=5, inputs=[])]
    with pytest.raises(rt.RtossError):
        rt.rtoss_group_layers(bad)


def test_create_fails_loudly_without_a_device(rt):
    import torch
    if torch.cuda.is_available():
        pytest.skip("a CUDA device is present")
    with pytest.raises(rt.RtossError):
        rt.Context(0)


def test_retinanet_program_add_fusion_keeps_a_valid_order():
    """Host logic of the chained RetinaNet-shaped runner: every add fed by an activation-free convolution that
    nothing else reads is folded into that convolution (16 block ends, 2 pyramid sums), each buffer is still
    written before it is read, and the same buffers are produced."""
    from paper_2303_02191_b200 import retinanet_net as rn
    ops, bufs, layers, outs = rn.program(800, 1088)
    fused = rn.fuse_adds(ops, outs)
    assert sum(op[0] == "add" for op in ops) == 18
    assert sum(op[0] == "convres" for op in fused) == 18 and not any(op[0] == "add" for op in fused)
    assert len(fused) == len(ops) - 18
    assert sorted(op[1] for op in fused if op[0] in ("conv", "convres")) == list(range(100))
    written = {"in"}
    for op in fused:
        srcs = op[2:3] if op[0] == "conv" else (op[2], op[4]) if op[0] == "convres" else op[1:2]
        dst = op[3] if op[0] == "conv" else op[5] if op[0] == "convres" else op[2]
        assert all(s in written for s in srcs), op
        assert dst not in written
        written.add(dst)
        if op[0] == "convres":
            assert bufs[op[3]] == bufs[op[4]] == bufs[op[5]]
            assert op[3] not in written
    assert all(o in written for o in outs)
    original = {op[3] if op[0] in ("conv", "add") else op[2] for op in ops}
    skipped = {op[3] for op in fused if op[0] == "convres"}
    assert written - {"in"} == original - skipped


def test_pattern_rank_matches_the_oracle_on_ties_and_cuts(rt):
    """rtoss_pattern_rank is host code: counts with many ties, every cut size."""
    rng = np.random.default_rng(3)
    for k, preset in ((2, orc.PRESET_CONN4), (3, orc.PRESET_CONN4), (4, orc.PRESET_ALL)):
        masks = orc.pattern_preset(k, preset)
        counts = rng.integers(0, 6, size=len(masks)).astype(np.uint64)     # few distinct values: many ties
        for M in (1, 2, len(masks) // 2, len(masks)):
            top, order = rt.rtoss_pattern_rank(masks, counts, k, M)
            want_top, want_order = orc.pattern_rank(masks, counts, M)
            assert np.array_equal(top, want_top) and np.array_equal(order, want_order)
    masks = orc.pattern_preset(2, orc.PRESET_CONN4)
    with pytest.raises(rt.RtossError):
        rt.rtoss_pattern_rank(masks, np.zeros(len(masks), dtype=np.uint64), 2, 0)
    with pytest.raises(rt.RtossError):
        rt.rtoss_pattern_rank(masks, np.zeros(len(masks), dtype=np.uint64), 2, len(masks) + 1)
    with pytest.raises(rt.RtossError):
        rt.rtoss_pattern_rank(masks, np.zeros(len(masks), dtype=np.uint64), 3, 2)      # table is not a 3-entry table
