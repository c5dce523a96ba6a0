"""Launch schedule of the chained network programs (host logic): rounds respect every producer -> consumer edge, a
buffer written in slices is ready only when all its slices are, and the tower layers of the RetinaNet-shaped program
fall into common rounds."""
from paper_2303_02191_b200 import retinanet_net, schedule, yolov5s_net


def _reads(op):
    if op[0] == "conv":
        return (op[2],)
    if op[0] == "add":
        return (op[1], op[2])
    return (op[1],)


def test_rounds_respect_dependencies_yolov5s():
    ops, bufs, layers = yolov5s_net.program(640, 640)
    write = lambda op: op[{"conv": 3, "add": 3, "pool5": 2, "up": 2, "copy": 2}[op[0]]]
    rounds = schedule.levels(ops, _reads, write, late=False)
    at = {i: r for r, idx in enumerate(rounds) for i in idx}
    assert sorted(at) == list(range(len(ops)))
    for i, op in enumerate(ops):
        for src in _reads(op):
            for j, other in enumerate(ops):
                if write(other) == src:
                    assert at[j] < at[i], (i, j)
    # the two 1x1 branches that open a C3 block read the same tensor: same round
    convs = {op[1]: i for i, op in enumerate(ops) if op[0] == "conv"}
    for a, b in ((2, 3), (8, 9), (16, 17), (26, 27), (34, 35), (40, 41), (46, 47), (52, 53)):
        assert at[convs[a]] == at[convs[b]]
    # cv3 of the first C3 block reads a concatenation written by a copy and by cv2: later than both
    assert at[convs[6]] > at[convs[3]]


def test_tower_layers_share_rounds_retinanet():
    ops, bufs, layers, outs = retinanet_net.program(800, 1088)
    write = lambda op: op[{"conv": 3, "add": 3, "up": 2, "relu": 2}[op[0]]]
    rounds = schedule.levels(ops, _reads, write)
    at = {i: r for r, idx in enumerate(rounds) for i in idx}
    conv_op = {op[1]: i for i, op in enumerate(ops) if op[0] == "conv"}
    # tower layer 0 on all five levels of both towers: one round (calls 60, 64, 68, 72, 76 and 80, 84, 88, 92, 96)
    assert len({at[conv_op[c]] for c in (60, 64, 68, 72, 76, 80, 84, 88, 92, 96)}) == 1
    for i, op in enumerate(ops):      # and every edge still points forward
        for src in _reads(op):
            for j, other in enumerate(ops):
                if write(other) == src:
                    assert at[j] < at[i], (i, j)
    # a tower layer follows the one before it on its own level
    for c in range(60, 100):
        if (c - 60) % 4:
            assert at[conv_op[c]] == at[conv_op[c - 1]] + 1
    assert max(len(r) for r in rounds) >= 8


def test_reading_before_writing_is_an_error():
    import pytest
    ops = [("conv", 0, "b", "c", 0), ("conv", 1, "a", "b", 0)]
    with pytest.raises(ValueError):
        schedule.levels(ops, lambda op: (op[2],), lambda op: op[3])


def test_chains_keep_program_order_and_every_edge():
    """schedule.chains: every operation is issued exactly once; an operation is issued after everything it reads;
    inside a shared launch the masks name exactly the producers that sit in the same launch."""
    ops, bufs, layers, outs = retinanet_net.program(800, 1088)
    ops = retinanet_net.fuse_adds(ops, outs)

    def reads(op):
        return (op[2], op[4]) if op[0] == "convres" else _reads(op)
    write = lambda op: op[{"conv": 3, "convres": 5, "add": 3, "up": 2, "relu": 2}[op[0]]]
    is_conv = lambda op: op[0] in ("conv", "convres")
    rounds = schedule.levels(ops, reads, write)
    steps = schedule.chains(ops, rounds, reads, write, is_conv)
    issued, written = [], set(["in"])
    for st in steps:
        idx = st[1] if st[0] == "chain" else [st[1]]
        if st[0] == "chain":
            assert 2 <= len(idx) <= 20 and all(is_conv(ops[i]) for i in idx)
            for q, i in enumerate(idx):
                want = 0
                for r in reads(ops[i]):
                    for p, j in enumerate(idx):
                        if write(ops[j]) == r:
                            assert p < q
                            want |= 1 << p
                assert st[2][q] == want
        for q, i in enumerate(idx):
            for r in reads(ops[i]):
                assert r in written or any(write(ops[j]) == r for j in idx[:q]), (i, r)
        for i in idx:
            written.add(write(ops[i]))
        issued += idx
    assert sorted(issued) == list(range(len(ops)))
    # successive tower layers end up in shared launches: far fewer steps than operations, and one launch of twenty
    assert max(len(st[1]) for st in steps if st[0] == "chain") == 20
    # a round of one convolution is never put into a shared launch
    for st in steps:
        if st[0] == "chain":
            lv = {i: r for r, rnd in enumerate(rounds) for i in rnd}
            for r in set(lv[i] for i in st[1]):
                assert sum(1 for i in st[1] if lv[i] == r) >= 2


def test_chained_units_of_the_retinanet_stack():
    from paper_2303_02191_b200 import synth
    layers = synth.retinanet_r50fpn_stack()
    units, afters = synth.chained_units(layers)
    assert sorted(i for u in units for i in u) == list(range(len(layers)))
    big = [(u, a) for u, a in zip(units, afters) if a is not None]
    assert [len(u) for u, _ in big] == [20, 20]
    for u, a in big:
        for q, i in enumerate(u):
            name = layers[i]["name"]
            tower, level = name.split(".")
            n = int(tower[-1])
            if n % 2 == 0:
                assert a[q] == 0
            else:
                (j,) = [p for p in range(len(u)) if (a[q] >> p) & 1]
                assert j < q and layers[u[j]]["name"] == "%s%d.%s" % (tower[:-1], n - 1, level)
    # every other unit is a set of independent convolutions, as before
    assert [u for u, a in zip(units, afters) if a is None] == [u for u in synth.independent_sets(layers) if "_tower" not in layers[u[0]]["name"]]
