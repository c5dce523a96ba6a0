"""RetinaNet ResNet-50-FPN-shaped network as ONE chained program over the library's calls.

The 100 pattern-pruned convolution calls of `synth.retinanet_r50fpn_stack()` (68 weight tensors: the two towers
share theirs across the five pyramid levels) plus the glue a whole network needs: the residual add + ReLU that
closes every bottleneck, the top-down pathway of the pyramid (2x up-sampling + add), the ReLU in front of P7.
The program starts at the 64-channel tensor behind the 7x7 stem and its max-pool (those are outside the 3x3 / 1x1
pattern set).  The same description drives `GpuNet` here (the C-ABI library, NHWC bf16, suitable for CUDA-graph
capture) and the tests' CPU-oracle executor.  Only shapes come from the model family; weights are seeded and
synthetic.
"""
from . import schedule, synth


def program(H0, W0):
    """-> (ops, bufs, layers).  bufs: name -> (C, H, W).  ops in execution order:
    ('conv', layer_index, src, dst, act) | ('add', a, b, dst, act) | ('up', src, dst) | ('relu', src, dst)."""
    layers = synth.retinanet_r50fpn_stack(H0, W0)
    ops, bufs = [], {}
    li = [0]

    def buf(name, C, H, W):
        bufs[name] = (C, H, W)
        return name

    def conv(src, dst, act):
        L = layers[li[0]]
        assert bufs[src] == (L["cin"], L["H"], L["W"]), (L["name"], bufs[src])
        Ho, Wo = synth.out_hw(L["H"], L["W"], L["stride"])
        assert bufs[dst] == (L["cout"], Ho, Wo), (L["name"], bufs[dst])
        ops.append(("conv", li[0], src, dst, act))
        li[0] += 1

    H, W = H0 // 4, W0 // 4
    cur = buf("in", 64, H, W)
    cin = 64
    feats = {}
    for si, (nblk, w) in enumerate(zip([3, 4, 6, 3], [64, 128, 256, 512])):
        for b in range(nblk):
            s = 2 if (b == 0 and si > 0) else 1
            tag = "layer%d.%d" % (si + 1, b)
            Ho, Wo = synth.out_hw(H, W, s)
            conv(cur, buf(tag + ".t1", w, H, W), "relu")
            conv(tag + ".t1", buf(tag + ".t2", w, Ho, Wo), "relu")
            conv(tag + ".t2", buf(tag + ".t3", 4 * w, Ho, Wo), "none")     # the ReLU comes after the residual add
            idn = cur
            if b == 0:
                conv(cur, buf(tag + ".idn", 4 * w, Ho, Wo), "none")
                idn = tag + ".idn"
            ops.append(("add", tag + ".t3", idn, buf(tag + ".out", 4 * w, Ho, Wo), "relu"))
            cur, cin, H, W = tag + ".out", 4 * w, Ho, Wo
        feats[si] = (cur, cin, H, W)
    # pyramid: laterals, top-down sums, 3x3 outputs, P6 from P5, P7 from ReLU(P6)
    for si in (1, 2, 3):
        src, c, h, w_ = feats[si]
        conv(src, buf("lat%d" % (si + 2), 256, h, w_), "none")
    for si in (2, 1):   # m5 = lat5; m4 = lat4 + up(m5); m3 = lat3 + up(m4)
        _, _, h, w_ = feats[si]
        top = "lat5" if si == 2 else "m4"
        ops.append(("up", top, buf("up%d" % (si + 2), 256, h, w_)))
        ops.append(("add", "lat%d" % (si + 2), "up%d" % (si + 2), buf("m%d" % (si + 2), 256, h, w_), "none"))
    levels = []
    for si in (1, 2, 3):
        _, _, h, w_ = feats[si]
        conv("lat5" if si == 3 else "m%d" % (si + 2), buf("p%d" % (si + 2), 256, h, w_), "none")
        levels.append(("p%d" % (si + 2), h, w_))
    _, h, w_ = levels[-1]
    h6, w6 = synth.out_hw(h, w_, 2)
    conv("p5", buf("p6", 256, h6, w6), "none")
    levels.append(("p6", h6, w6))
    ops.append(("relu", "p6", buf("p6.relu", 256, h6, w6)))
    h7, w7 = synth.out_hw(h6, w6, 2)
    conv("p6.relu", buf("p7", 256, h7, w7), "none")
    levels.append(("p7", h7, w7))
    outputs = []
    for tower in ("cls", "box"):
        for (feat, h, w_) in levels:
            src = feat
            for i in range(4):
                dst = buf("%s.%s.%d" % (tower, feat, i), 256, h, w_)
                conv(src, dst, "relu")
                src = dst
            outputs.append(src)
    assert li[0] == len(layers) == 100
    return ops, bufs, layers, tuple(outputs)


def fuse_adds(ops, outputs):
    """Every 'add' one of whose operands comes from a convolution without activation and is read by nothing else
    becomes ('convres', layer_index, src, tmp, other, dst, act) at the add's place: the convolution moves there (each
    buffer of the program is written once, so moving a producer later changes nothing) and adds the other operand in
    its epilogue.  tmp is the buffer the convolution would have written, used when the fused call is declined."""
    reads = {}
    for op in ops:
        srcs = (op[2],) if op[0] == "conv" else (op[1], op[2]) if op[0] == "add" else (op[1],)
        for s_ in srcs:
            reads[s_] = reads.get(s_, 0) + 1
    for name in outputs:
        reads[name] = reads.get(name, 0) + 1
    producer = {op[3]: j for j, op in enumerate(ops) if op[0] == "conv" and op[4] == "none"}
    moved, out = {}, []
    for j, op in enumerate(ops):
        if op[0] == "add":
            for tmp, other in ((op[1], op[2]), (op[2], op[1])):
                if tmp in producer and reads[tmp] == 1 and tmp != other:
                    moved[producer[tmp]] = ("convres", ops[producer[tmp]][1], ops[producer[tmp]][2], tmp, other, op[3], op[4])
                    break
    by_add = {v[5]: v for v in moved.values()}
    for j, op in enumerate(ops):
        if j in moved:
            continue
        out.append(by_add[op[3]] if op[0] == "add" and op[3] in by_add else op)
    return out


class GpuNet:
    """The program on the GPU through the C-ABI library: NHWC, bf16 (or fp16), k-entry patterns."""

    def __init__(self, ctx, N, H0=800, W0=1088, k=4, seed=0, dtype="bf16", fuse_residual=True):
        import torch
        from . import binding as rt
        self.rt, self.ctx, self.N, self.torch = rt, ctx, N, torch
        self.ops, self.bufs, self.layers, self.output_names = program(H0, W0)
        if fuse_residual:
            self.ops = fuse_adds(self.ops, self.output_names)
        self.unfused = set()   # layers whose fused call the library declined: convolution and add run separately
        self.rounds, self.probed, self.steps = None, False, None
        tdt = {"bf16": torch.bfloat16, "f16": torch.float16}[dtype]
        self.t = {n: torch.zeros((N, H, W, C), dtype=tdt, device="cuda") for n, (C, H, W) in self.bufs.items()}
        self.zero = {}   # all-zero operands of the ReLU glue op, one per shape
        for op in self.ops:
            if op[0] == "relu" and self.bufs[op[1]] not in self.zero:
                C, H, W = self.bufs[op[1]]
                self.zero[self.bufs[op[1]]] = torch.zeros((N, H, W, C), dtype=tdt, device="cuda")
        masks = rt.rtoss_pattern_preset(k, rt.PRESET_CENTRE8 if k == 4 else rt.PRESET_CONN4)
        self.packed, self.bias = {}, {}
        for L in self.layers:
            if L["wid"] in self.packed:
                continue
            w = torch.from_numpy(synth.kaiming_weights(seed, 3000 + L["wid"], L["cout"], L["cin"], L["ksize"])).cuda()
            pid = ctx.rtoss_select_patterns(w, L["ksize"], masks, k)
            self.packed[L["wid"]] = ctx.rtoss_pack(w, L["ksize"], masks, k, pid, rt.DTYPE_NAMES[dtype])
            self.bias[L["wid"]] = torch.from_numpy(synth.bias(seed, 3000 + L["wid"], L["cout"])).cuda()
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
        return op[{"conv": 3, "convres": 5, "add": 3, "up": 2, "relu": 2}[op[0]]]

    def run(self, grouped=True, chained=False):
        """One pass.  grouped: operations are issued round by round (schedule.levels) and the convolutions of a round go
        out through rtoss_conv_group; else one call per operation in program order."""
        self.launches = 0      # kernel launches of this pass
        if not grouped or not self.probed:
            for op in self.ops:
                self._run_op(op)
            self.probed = True     # the first pass finds out which fused residual calls the library declines
            return
        if self.rounds is None:
            # as late as possible: tower layer i of every pyramid level then shares a round (and a launch)
            self.rounds = schedule.levels(self.ops, self._reads, self._write, late=True)
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
            convs = [self.ops[i] for i in rnd if self.ops[i][0] == "conv" or (self.ops[i][0] == "convres" and self.ops[i][1] not in self.unfused)]
            rest = [self.ops[i] for i in rnd if not (self.ops[i][0] == "conv" or (self.ops[i][0] == "convres" and self.ops[i][1] not in self.unfused))]
            if len(convs) >= 2:
                self.launches += self.ctx.rtoss_conv_group([self._item(op) for op in convs])
            else:
                rest = convs + rest
            for op in rest:
                self._run_op(op)

    def _item(self, op):
        rt, N, t = self.rt, self.N, self.t
        L = self.layers[op[1]]
        if op[0] == "conv":
            _, i, src, dst, act = op
            return self.ctx.conv_item(self.packed[L["wid"]], t[src], t[dst], N, L["H"], L["W"], L["stride"], rt.NHWC, rt.ACT_NAMES[act],
                                      self.bias[L["wid"]])
        _, i, src, tmp, other, dst, act = op
        return self.ctx.conv_item(self.packed[L["wid"]], t[src], t[dst], N, L["H"], L["W"], L["stride"], rt.NHWC, rt.ACT_NAMES[act],
                                  self.bias[L["wid"]], residual=t[other])

    def _run_op(self, op):
        rt, N, t = self.rt, self.N, self.t
        self.launches += 1
        if op[0] == "conv":
            _, i, src, dst, act = op
            L = self.layers[i]
            fn = self.ctx.rtoss_conv3x3_pattern if L["ksize"] == 3 else self.ctx.rtoss_conv1x1_pattern
            fn(self.packed[L["wid"]], t[src], t[dst], N, L["H"], L["W"], L["stride"], rt.NHWC, rt.ACT_NAMES[act],
               self.bias[L["wid"]])
        elif op[0] == "convres":   # convolution (no activation) + residual + activation in one call
            _, i, src, tmp, other, dst, act = op
            L = self.layers[i]
            fn = self.ctx.rtoss_conv3x3_pattern if L["ksize"] == 3 else self.ctx.rtoss_conv1x1_pattern
            args = (self.packed[L["wid"]], t[src], None, N, L["H"], L["W"], L["stride"], rt.NHWC)
            if i not in self.unfused:
                try:
                    fn(*args[:2], t[dst], *args[3:], rt.ACT_NAMES[act], self.bias[L["wid"]], residual=t[other])
                    return
                except rt.RtossError as err:
                    if err.status != rt.ERR_UNSUPPORTED:
                        raise
                    self.unfused.add(i)
                    self.rounds = self.steps = None
            fn(*args[:2], t[tmp], *args[3:], rt.ACT_NONE, self.bias[L["wid"]])
            rt.rtoss_add_act(t[tmp], t[other], t[dst], rt.ACT_NAMES[act])
            self.launches += 1
        elif op[0] == "add":
            rt.rtoss_add_act(t[op[1]], t[op[2]], t[op[3]], rt.ACT_NAMES[op[4]])
        elif op[0] == "up":
            C, H, W = self.bufs[op[1]]
            rt.rtoss_upsample2x(t[op[1]], t[op[2]], N, C, H, W, rt.NHWC)
        elif op[0] == "relu":
            rt.rtoss_add_act(t[op[1]], self.zero[self.bufs[op[1]]], t[op[2]], rt.ACT_RELU)

    def outputs(self):
        return {n: self.t[n].float().permute(0, 3, 1, 2).cpu().numpy() for n in self.output_names}

    def close(self):
        for p in self.packed.values():
            p.close()
