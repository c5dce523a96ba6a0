"""Wiring of the two chained network programs against hand-made tables of the architectures
(`tests/golden/yolov5s_wiring.txt`, `tests/golden/retinanet_wiring.txt`): for every convolution the expression
that feeds it (which convolutions, through which adds / pools / up-samplings, concatenated in which order), its
shape, stride and -- for the RetinaNet-shaped towers -- which calls share a weight tensor.  The chained parity
tests execute the same `program()` on both sides, so a mis-wired edge or a wrong concatenation offset would pass
them unseen; here the program is compared with a description it was not generated from."""
import os
import re

from paper_2303_02191_b200 import retinanet_net, synth, yolov5s_net

GOLDEN = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden")


def _read(name, n_fields):
    defs, rows, outputs = {}, [], None
    for line in open(os.path.join(GOLDEN, name)):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        if line.startswith("outputs ="):
            outputs = line.split("=", 1)[1].split()
        elif "|" in line:
            f = [v.strip() for v in line.split("|", n_fields - 1)]
            assert len(f) == n_fields, line
            rows.append(f)
        else:
            k, v = [s.strip() for s in line.split("=", 1)]
            defs[k] = v
    return defs, rows, outputs


def _expand(expr, defs):
    """Replace shorthands by their definitions until none is left; sums are commutative: operands sorted."""
    for _ in range(64):
        new = re.sub(r"\b([a-z]+[0-9]*_?[0-9]*)\b", lambda m: defs.get(m.group(1), m.group(1)), expr)
        if new == expr:
            break
        expr = new
    return _canon(expr)


def _split_top(s, sep):
    out, depth, cur = [], 0, ""
    for ch in s:
        if ch == "(":
            depth += 1
        elif ch == ")":
            depth -= 1
        if ch == sep and depth == 0:
            out.append(cur)
            cur = ""
        else:
            cur += ch
    out.append(cur)
    return out


def _canon(e):
    e = e.strip()
    m = re.match(r"^([a-z]+)\((.*)\)$", e)
    if not m or len(_split_top(e, "|")) > 1 and not e.startswith("cat("):
        return e
    fn, inner = m.group(1), m.group(2)
    # the match must close at the end: "add(a,b)" yes, "up(a)|b" no
    depth = 0
    for i, ch in enumerate(e):
        depth += ch == "("
        depth -= ch == ")"
        if depth == 0 and ch == ")" and i != len(e) - 1:
            return e
    if fn == "cat":
        return "cat(" + "|".join(_canon(p) for p in _split_top(inner, "|")) + ")"
    if fn == "add":
        return "add(" + ",".join(sorted(_canon(p) for p in _split_top(inner, ","))) + ")"
    return fn + "(" + _canon(inner) + ")"


def test_yolov5s_program_matches_the_hand_made_wiring_table():
    defs, rows, outputs = _read("yolov5s_wiring.txt", 6)
    ops, bufs, layers = yolov5s_net.program(640, 640)
    assert len(rows) == len(layers) == 57
    assert [op[1] for op in ops if op[0] == "conv"] == list(range(57))
    held, reads, value = _trace_incremental(ops, bufs, layers, "yolo")
    for f in rows:
        i = int(f[0])
        L = layers[i]
        assert (L["ksize"], L["stride"], L["cin"], L["cout"]) == tuple(int(v) for v in f[1:5]), "layer %d shape" % i
        assert _canon(reads[i]) == _expand(f[5], defs), "convolution %d reads %s" % (i, reads[i])
    assert [_canon(value(n)) for n in yolov5s_net.OUTPUTS] == [_expand(o, defs) for o in outputs]
    # resolutions: 640 -> 320 -> 160 -> 80 -> 40 -> 20, the neck back up to 80 and down again
    want_hw = {0: 640, 1: 320, 2: 160, 7: 160, 8: 80, 15: 80, 16: 40, 25: 40, 26: 20, 33: 20, 34: 40, 39: 40, 40: 80, 45: 80,
               46: 40, 51: 40, 52: 20}
    for i, hw in want_hw.items():
        assert (layers[i]["H"], layers[i]["W"]) == (hw, hw), i


def _trace_incremental(ops, bufs, layers, kind):
    """_trace with the channel count of a convolution's output taken from the layer table."""
    held = {"in": {0: (bufs["in"][0], "in")}}
    reads = {}

    def value(name):
        parts = sorted(held[name].items())
        total = sum(c for _, (c, _) in parts)
        assert total == bufs[name][0], "buffer %s is read with %d of its %d channels written" % (name, total, bufs[name][0])
        at = 0
        for off, (c, _) in parts:
            assert off == at, "buffer %s: slices overlap or leave a gap at channel %d" % (name, at)
            at += c
        return parts[0][1][1] if len(parts) == 1 else "cat(" + "|".join(e for _, (_, e) in parts) + ")"

    def write(name, off, C, expr):
        held.setdefault(name, {})
        assert off not in held[name], "buffer %s slice %d written twice" % (name, off)
        held[name][off] = (C, expr)

    for op in ops:
        if op[0] == "conv":
            i, src, dst = op[1], op[2], op[3]
            L = layers[i]
            assert bufs[src][0] == L["cin"] and bufs[src][1:] == (L["H"], L["W"]), "convolution %d input shape" % i
            Ho, Wo = synth.out_hw(L["H"], L["W"], L["stride"])
            assert bufs[dst][1:] == (Ho, Wo), "convolution %d output size" % i
            reads[i] = value(src)
            write(dst, op[4] if kind == "yolo" else 0, L["cout"], "c%d" % i)
        elif op[0] == "add":
            assert bufs[op[1]] == bufs[op[2]] == bufs[op[3]]
            e = "add(%s,%s)" % (value(op[1]), value(op[2]))
            if kind == "retina" and op[4] == "relu":
                e = "relu(%s)" % e
            write(op[3], 0, bufs[op[3]][0], e)
        elif op[0] == "pool5":
            assert bufs[op[1]][1:] == bufs[op[2]][1:]
            write(op[2], op[3], bufs[op[1]][0], "pool(%s)" % value(op[1]))
        elif op[0] == "up":
            assert (2 * bufs[op[1]][1], 2 * bufs[op[1]][2]) == bufs[op[2]][1:]
            write(op[2], op[3] if kind == "yolo" else 0, bufs[op[1]][0], "up(%s)" % value(op[1]))
        elif op[0] == "copy":
            assert bufs[op[1]][1:] == bufs[op[2]][1:]
            write(op[2], op[3], bufs[op[1]][0], value(op[1]))
        elif op[0] == "relu":
            write(op[2], 0, bufs[op[1]][0], "relu(%s)" % value(op[1]))
        else:
            raise AssertionError("unknown op " + op[0])
    return held, reads, value


def test_retinanet_program_matches_the_wiring_table():
    defs, rows, outputs = _read("retinanet_wiring.txt", 8)
    ops, bufs, layers, outs = retinanet_net.program(800, 1088)
    assert len(rows) == len(layers) == 100
    held, reads, value = _trace_incremental(ops, bufs, layers, "retina")
    acts = {op[1]: op[4] for op in ops if op[0] == "conv"}
    wid_of = {}
    for f in rows:
        i = int(f[0])
        L = layers[i]
        assert (L["ksize"], L["stride"], L["cin"], L["cout"]) == tuple(int(v) for v in f[1:5]), "call %d shape" % i
        assert acts[i] == f[5], "call %d activation" % i
        wid_of.setdefault(f[6], set()).add(L["wid"])
        assert _canon(reads[i]) == _expand(f[7], defs), "call %d reads %s" % (i, reads[i])
    # the table's weight names and the program's weight ids are the same partition of the calls
    assert all(len(v) == 1 for v in wid_of.values())
    assert len({next(iter(v)) for v in wid_of.values()}) == len(wid_of) == 68
    assert [_canon(value(n)) for n in outs] == [_expand(o, defs) for o in outputs]
    # pyramid resolutions for an 800 x 1088 frame
    sizes = {52: (100, 136), 53: (50, 68), 54: (25, 34), 58: (25, 34), 59: (13, 17), 76: (7, 9), 96: (7, 9)}
    for i, hw in sizes.items():
        assert (layers[i]["H"], layers[i]["W"]) == hw, i


def test_the_tracer_notices_a_wrong_offset_and_a_swapped_edge():
    """The comparison itself: a concatenation offset moved, or an edge re-pointed, must change what is read."""
    ops, bufs, layers = yolov5s_net.program(640, 640)
    _, good, _ = _trace_incremental(ops, bufs, layers, "yolo")
    bad = list(ops)
    j = next(i for i, op in enumerate(bad) if op[0] == "copy" and op[2] == "n.cat1")
    bad[j] = ("copy", "p3", "n.cat1", 256) if bufs["p3"] == bufs["p4"] else ("copy", "p4", "n.cat1", 0)
    try:
        _, reads, _ = _trace_incremental(bad, bufs, layers, "yolo")
        changed = reads != good
    except AssertionError:
        changed = True
    assert changed
