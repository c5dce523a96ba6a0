"""YOLOv5s-shaped backbone + neck as ONE chained program over the library's calls.

The 57 pattern-pruned convolutions of `synth.yolov5s_stack()` plus the glue a whole network needs
(residual adds, SPPF max-pooling, up-sampling, concatenations as channel-slice writes).  The same
description drives `GpuNet` here (the C-ABI library, NHWC bf16, suitable for CUDA-graph capture) and
the tests' CPU-oracle executor used for the chained parity check on small inputs.
Only shapes come from the model family; weights are seeded and synthetic.
"""
import numpy as np

from . import schedule, synth


def program(H0, W0):
    """-> (ops, buffers).  buffers: name -> (C, H, W).  ops in execution order:
    ('conv', layer_index, src, dst, dst_channel_offset) | ('add', a, b, dst) | ('pool5', src, dst, off) (5x5, stride 1) |
    ('up', src, dst, off) | ('copy', src, dst, off)."""
    layers = synth.yolov5s_stack(H0, W0)
    ops, bufs = [], {}
    li = [0]

    def buf(name, C, H, W):
        bufs[name] = (C, H, W)
        return name

    def conv(src, dst, off=0):
        ops.append(("conv", li[0], src, dst, off))
        li[0] += 1

    def c3(tag, src, c2, n, shortcut, H, W, out):
        h = c2 // 2
        cat = buf(tag + ".cat", c2, H, W)
        a = buf(tag + ".a", h, H, W)
        conv(src, a)                     # cv1
        conv(src, cat, h)                # cv2 -> second half of the concatenation
        cur = a
        for i in range(n):
            t1 = buf("%s.m%d.t1" % (tag, i), h, H, W)
            conv(cur, t1)
            last = i == n - 1
            if shortcut:
                t2 = buf("%s.m%d.t2" % (tag, i), h, H, W)
                conv(t1, t2)
                nxt = buf("%s.m%d.out" % (tag, i), h, H, W)
                ops.append(("add", cur, t2, nxt))
                cur = nxt
                if last:
                    ops.append(("copy", cur, cat, 0))
            elif last:
                conv(t1, cat, 0)         # straight into the first half of the concatenation
            else:
                t2 = buf("%s.m%d.t2" % (tag, i), h, H, W)
                conv(t1, t2)
                cur = t2
        conv(cat, out)                   # cv3

    H, W = H0, W0
    buf("in", 3, H, W)
    H, W = synth.out_hw(H, W, 2); conv("in", buf("s0", 32, H, W))
    H, W = synth.out_hw(H, W, 2); conv("s0", buf("s1", 64, H, W))
    c3("c3_1", "s1", 64, 1, True, H, W, buf("b1", 64, H, W))
    H, W = synth.out_hw(H, W, 2); conv("b1", buf("s2", 128, H, W)); H8, W8 = H, W
    c3("c3_2", "s2", 128, 2, True, H, W, buf("p3", 128, H, W))
    H, W = synth.out_hw(H, W, 2); conv("p3", buf("s3", 256, H, W)); H16, W16 = H, W
    c3("c3_3", "s3", 256, 3, True, H, W, buf("p4", 256, H, W))
    H, W = synth.out_hw(H, W, 2); conv("p4", buf("s4", 512, H, W)); H32, W32 = H, W
    c3("c3_4", "s4", 512, 1, True, H, W, buf("b4", 512, H, W))
    # SPPF: 1x1, three chained 5x5 max-pools, concatenation of the four, 1x1
    buf("sppf.cat", 1024, H, W)
    conv("b4", buf("sppf.m0", 256, H, W))
    ops.append(("copy", "sppf.m0", "sppf.cat", 0))
    for i in range(3):
        ops.append(("pool5", "sppf.m%d" % i, buf("sppf.m%d" % (i + 1), 256, H, W), 0))
        ops.append(("copy", "sppf.m%d" % (i + 1), "sppf.cat", 256 * (i + 1)))
    conv("sppf.cat", buf("p5", 512, H, W))
    # neck, top-down
    buf("n.cat1", 512, H16, W16)
    conv("p5", buf("n1", 256, H32, W32))
    ops.append(("up", "n1", "n.cat1", 0))
    ops.append(("copy", "p4", "n.cat1", 256))
    c3("n.c3_1", "n.cat1", 256, 1, False, H16, W16, buf("t4", 256, H16, W16))
    buf("n.cat2", 256, H8, W8)
    conv("t4", buf("n2", 128, H16, W16))
    ops.append(("up", "n2", "n.cat2", 0))
    ops.append(("copy", "p3", "n.cat2", 128))
    c3("n.c3_2", "n.cat2", 128, 1, False, H8, W8, buf("o3", 128, H8, W8))
    # bottom-up
    buf("n.cat3", 256, H16, W16)
    conv("o3", "n.cat3", 0)
    ops.append(("copy", "n2", "n.cat3", 128))
    c3("n.c3_3", "n.cat3", 256, 1, False, H16, W16, buf("o4", 256, H16, W16))
    buf("n.cat4", 512, H32, W32)
    conv("o4", "n.cat4", 0)
    ops.append(("copy", "n1", "n.cat4", 256))
    c3("n.c3_4", "n.cat4", 512, 1, False, H32, W32, buf("o5", 512, H32, W32))
    assert li[0] == len(layers) == 57
    return ops, bufs, layers


OUTPUTS = ("o3", "o4", "o5")


def fuse_shortcuts(ops):
    """A bottleneck's shortcut add directly behind its second convolution, whose output nothing else reads, becomes
    ('convres', layer_index, src, tmp, other, dst): the convolution adds the block input behind its activation."""
    reads = {}
    for op in ops:
        for s_ in ((op[2],) if op[0] == "conv" else (op[1], op[2]) if op[0] == "add" else (op[1],)):
            reads[s_] = reads.get(s_, 0) + 1
    out = []
    for op in ops:
        prev = out[-1] if out else None
        if (op[0] == "add" and prev is not None and prev[0] == "conv" and prev[4] == 0 and prev[3] == op[2]
                and reads[op[2]] == 1 and op[1] != op[2]):
            out[-1] = ("convres", prev[1], prev[2], prev[3], op[1], op[3])
        else:
            out.append(op)
    return out


class GpuNet:
    """The program on the GPU through the C-ABI library: NHWC, bf16 (or fp16), k-entry patterns."""

    def __init__(self, ctx, N, H0=640, W0=640, k=4, seed=0, dtype="bf16", fuse_residual=True):
        import torch
        from . import binding as rt
        self.rt, self.ctx, self.N, self.torch = rt, ctx, N, torch
        self.ops, self.bufs, self.layers = program(H0, W0)
        if fuse_residual:
            self.ops = fuse_shortcuts(self.ops)
        self.unfused = set()   # layers whose fused call the library declined: convolution and add run separately
        self.rounds, self.probed, self.steps = None, False, None
        tdt = {"bf16": torch.bfloat16, "f16": torch.float16}[dtype]
        self.t = {n: torch.zeros((N, H, W, C), dtype=tdt, device="cuda") for n, (C, H, W) in self.bufs.items()}
        masks = rt.rtoss_pattern_preset(k, rt.PRESET_CENTRE8 if k == 4 else rt.PRESET_CONN4)
        self.packed, self.bias = [], []
        for i, L in enumerate(self.layers):
            w = torch.from_numpy(synth.kaiming_weights(seed, 2000 + i, L["cout"], L["cin"], L["ksize"])).cuda()
            pid = ctx.rtoss_select_patterns(w, L["ksize"], masks, k)
            self.packed.append(ctx.rtoss_pack(w, L["ksize"], masks, k, pid, rt.DTYPE_NAMES[dtype]))
            self.bias.append(torch.from_numpy(synth.bias(seed, 2000 + i, L["cout"])).cuda())
        torch.cuda.synchronize()

    def set_input(self, x_nchw):
        self.t["in"].copy_(self.torch.from_numpy(x_nchw).permute(0, 2, 3, 1).to(self.t["in"].dtype))

    def _reads(self, op):
        if op[0] == "conv":
            return (op[2],)
        if op[0] == "convres":
            return (op[2], op[4])
        if op[0] == "add":
            return (op[1], op[2])
        return (op[1],)

    def _write(self, op):
        return op[{"conv": 3, "convres": 5, "add": 3, "pool5": 2, "up": 2, "copy": 2}[op[0]]]

    def run(self, grouped=True, chained=False):
        """One pass.  grouped: operations are issued round by round (schedule.levels: a buffer is ready when every slice
        of it has been written) and the convolutions of a round go out through rtoss_conv_group; else one call per
        operation in program order."""
        self.launches = 0      # kernel launches of this pass
        if not grouped or not self.probed:
            for op in self.ops:
                self._run_op(op)
            self.probed = True     # the first pass finds out which fused shortcut calls the library declines
            return
        if self.rounds is None:
            # as soon as possible: the two 1x1 branches that open a C3 block then share a round (and a launch)
            self.rounds = schedule.levels(self.ops, self._reads, self._write, late=False)
        is_conv_op = lambda op: op[0] == "conv" or (op[0] == "convres" and op[1] not in self.unfused)
        if chained:
            # convolutions of consecutive rounds go out together (rtoss_conv_chain: dependent convolutions in one launch)
            if self.steps is None:
                self.steps = schedule.chains(self.ops, self.rounds, self._reads, self._write, is_conv_op)
            for step in self.steps:
                if step[0] == "chain":
                    items = [self._item(self.ops[i]) for i in step[1]]
                    # (a segment without a dependency in it is a set of independent convolutions, as in the grouped run)
                    self.launches += self.ctx.rtoss_conv_chain(items, step[2]) if any(step[2]) else self.ctx.rtoss_conv_group(items)
                else:
                    self._run_op(self.ops[step[1]])
            return
        for rnd in self.rounds:
            is_conv = lambda op: op[0] == "conv" or (op[0] == "convres" and op[1] not in self.unfused)
            convs = [self.ops[i] for i in rnd if is_conv(self.ops[i])]
            rest = [self.ops[i] for i in rnd if not is_conv(self.ops[i])]
            if len(convs) >= 2:
                self.launches += self.ctx.rtoss_conv_group([self._item(op) for op in convs])
            else:
                rest = convs + rest
            for op in rest:
                self._run_op(op)

    def _item(self, op):
        rt, N, t = self.rt, self.N, self.t
        i = op[1]
        L = self.layers[i]
        if op[0] == "conv":
            _, _, src, dst, off = op
            return self.ctx.conv_item(self.packed[i], t[src], t[dst], N, L["H"], L["W"], L["stride"], rt.NHWC, rt.ACT_SILU, self.bias[i],
                                      off, self.bufs[dst][0])
        _, _, src, tmp, other, dst = op
        return self.ctx.conv_item(self.packed[i], t[src], t[dst], N, L["H"], L["W"], L["stride"], rt.NHWC, rt.ACT_SILU, self.bias[i],
                                  residual=t[other], residual_after_act=True)

    def _run_op(self, op):
        rt, N, t = self.rt, self.N, self.t
        self.launches += 1
        if op[0] == "conv":
            _, i, src, dst, off = op
            L = self.layers[i]
            fn = self.ctx.rtoss_conv3x3_pattern if L["ksize"] == 3 else self.ctx.rtoss_conv1x1_pattern
            fn(self.packed[i], t[src], t[dst], N, L["H"], L["W"], L["stride"], rt.NHWC, rt.ACT_SILU, self.bias[i],
               off, self.bufs[dst][0])
        elif op[0] == "convres":   # second convolution of a bottleneck + its shortcut in one call
            _, i, src, tmp, other, dst = op
            L = self.layers[i]
            fn = self.ctx.rtoss_conv3x3_pattern if L["ksize"] == 3 else self.ctx.rtoss_conv1x1_pattern
            if i not in self.unfused:
                try:
                    fn(self.packed[i], t[src], t[dst], N, L["H"], L["W"], L["stride"], rt.NHWC, rt.ACT_SILU, self.bias[i],
                       residual=t[other], residual_after_act=True)
                    return
                except rt.RtossError as err:
                    if err.status != rt.ERR_UNSUPPORTED:
                        raise
                    self.unfused.add(i)
                    self.rounds = self.steps = None
            fn(self.packed[i], t[src], t[tmp], N, L["H"], L["W"], L["stride"], rt.NHWC, rt.ACT_SILU, self.bias[i])
            rt.rtoss_add_act(t[other], t[tmp], t[dst], rt.ACT_NONE)
            self.launches += 1
        elif op[0] == "add":
            rt.rtoss_add_act(t[op[1]], t[op[2]], t[op[3]], rt.ACT_NONE)
        elif op[0] == "pool5":
            C, H, W = self.bufs[op[1]]
            rt.rtoss_maxpool2d(t[op[1]], t[op[2]], N, C, H, W, 5, 1, 2, rt.NHWC, op[3], self.bufs[op[2]][0])
        elif op[0] == "up":
            C, H, W = self.bufs[op[1]]
            rt.rtoss_upsample2x(t[op[1]], t[op[2]], N, C, H, W, rt.NHWC, op[3], self.bufs[op[2]][0])
        elif op[0] == "copy":
            C, H, W = self.bufs[op[1]]
            rt.rtoss_maxpool2d(t[op[1]], t[op[2]], N, C, H, W, 1, 1, 0, rt.NHWC, op[3], self.bufs[op[2]][0])

    def outputs(self):
        return {n: self.t[n].float().permute(0, 3, 1, 2).cpu().numpy() for n in OUTPUTS}

    def close(self):
        for p in self.packed:
            p.close()
