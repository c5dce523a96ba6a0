#!/usr/bin/env python
"""Benchmark of the R-TOSS hot path on B200.

A step is one pass of the whole hot path over one batch of synthetic input:
pattern selection (Algorithm 2 / 3 of arXiv 2303.02191), packing, and the
pattern-sparse convolution, for each layer of the workload.  Default workload
"retinanet_b4": the RetinaNet ResNet-50-FPN-shaped stack (100 convolution calls
on 68 weight tensors behind the 7x7 stem), batch 4 of 800x1088 frames, bf16,
4-entry patterns -- the largest configuration that fits one GPU.  The smaller
configurations ("layer32", "layer128", "yolov5s_b1", "yolov5s_b16") are measured
in the same run with fewer steps and reported as sub-records under "others".
Prints ONE JSON line (rank 0).  `--impl reference` times the CPU oracle instead.
"""
import argparse
import json
import os
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2303_02191_b200 import synth  # noqa: E402

# nominal FP32 FMA peak: 148 SMs x 128 lanes x 2 FLOP x 1.965 GHz (maximum SM clock)
ALU_PEAK_TFLOPS = 148 * 128 * 2 * 1.965e9 / 1e12


def workload_layers(name):
    """-> (batch N, dtype, list of (layer dict, k, preset name))."""
    if name == "layer128":
        l3 = dict(name="conv3x3_128", ksize=3, stride=1, cin=128, cout=128, H=80, W=80, act="silu", wid=0)
        l1 = dict(name="conv1x1_256_128", ksize=1, stride=1, cin=256, cout=128, H=80, W=80, act="silu", wid=2)
        return 8, "bf16", [(l3, 3, "conn4"), (dict(l3, wid=1), 2, "conn4"), (l1, 3, "conn4")]
    if name == "layer32":
        l3 = dict(name="conv3x3_32", ksize=3, stride=1, cin=32, cout=32, H=32, W=32, act="none", wid=0)
        return 1, "f32", [(l3, 4, "centre8")]
    if name in ("yolov5s_b1", "yolov5s_b16"):
        return (1 if name.endswith("b1") else 16), "bf16", [(L, 4, "centre8") for L in synth.yolov5s_stack()]
    if name == "retinanet_b4":
        return 4, "bf16", [(L, 4, "centre8") for L in synth.retinanet_r50fpn_stack()]
    if name == "retinanet_tower":
        # the launch that dominates retinanet_b4: the first two layers of both towers on the five pyramid levels
        return 4, "bf16", [(L, 4, "centre8") for L in synth.retinanet_r50fpn_stack() if "_tower0." in L["name"] or "_tower1." in L["name"]]
    raise SystemExit("unknown workload " + name)


# DRAM bytes per launch (dram__bytes_read.sum + dram__bytes_write.sum) of a workload's dominant kernel from one
# ncu capture (caches flushed before every pass; the command is recorded with the capture's summary), valid
# for the kernel source whose hash is recorded with it: once conv_tc.cu changes the figure is withheld (null).
# The launch is the first two layers of both RetinaNet towers on the five pyramid levels (twenty convolutions, the
# second ten waiting inside the kernel for the first ten), captured in the retinanet_tower workload, which issues
# exactly that launch: 151.5 MB read (the inputs of layer 0 and the weights once; half of layer 1's input, which
# layer 0 wrote a moment before, is still in the 126 MB L2) + 107.3 MB written.
NCU_TRAFFIC = {("retinanet_b4", "cls_tower0.p3+19", 4): (258770000, "f9cc1280503be3b1"),
               ("retinanet_tower", "cls_tower0.p3+19", 4): (258770000, "f9cc1280503be3b1")}


def ncu_traffic(workload, layer, k):
    import hashlib
    rec = NCU_TRAFFIC.get((workload, layer, k))
    if not rec:
        return None
    try:
        src = os.path.join(ROOT, "paper_2303_02191_b200", "csrc", "conv_tc.cu")
        if hashlib.sha256(open(src, "rb").read()).hexdigest()[:16] != rec[1]:
            return None
    except OSError:
        return None
    return rec[0]


def read_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        try:
            d = json.load(open(path))
            return float(d["hbm_gbs"]), float(d["bf16_tflops_sustained"]), "measured"
        except Exception:
            pass
    return 6650.0, 1400.0, "fallback"


class ClockSampler(threading.Thread):
    """Samples SM clock and throttle reasons through NVML while the timed region runs."""

    def __init__(self, index):
        super().__init__(daemon=True)
        self.index = index
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self._stop_evt = threading.Event()
        self.ok = False
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM)
            self.ok = True
        except Exception:
            self.ok = False

    def run(self):
        if not self.ok:
            return
        nv = self.nv
        names = {"hw_slowdown": 0x8, "sw_power_cap": 0x4, "sw_thermal_slowdown": 0x20, "hw_thermal_slowdown": 0x40,
                 "hw_power_brake": 0x80}
        while not self._stop_evt.is_set():
            try:
                self.samples.append(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM))
                try:
                    r = nv.nvmlDeviceGetCurrentClocksEventReasons(self.h)
                except Exception:
                    r = nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h)
                for k, bit in names.items():
                    if r & bit:
                        self.reasons.add(k)
            except Exception:
                pass
            time.sleep(0.005)

    def stop(self):
        self._stop_evt.set()
        self.join(timeout=2)
        med = float(np.median(self.samples)) if self.samples else None
        return {"sm_mhz": med, "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons), "samples": len(self.samples)}


def physical_gpu_index(local_rank):
    vis = os.environ.get("CUDA_VISIBLE_DEVICES")
    if vis:
        try:
            return int(vis.split(",")[local_rank])
        except Exception:
            return local_rank
    return local_rank


# --------------------------------------------------------------------------- CPU oracle legs

_PREPARED = {}


def oracle_inputs(layers_k, dtype, n_sample, seed=0):
    """Seeded inputs of every layer for the oracle legs, generated once per (workload, sample size)."""
    key = (id(layers_k), dtype, n_sample, seed)
    if key not in _PREPARED:
        from oracle import rtoss_oracle as orc
        prepared = []
        for (L, k, preset) in layers_k:
            masks = orc.pattern_preset(k, orc.PRESET_CENTRE8 if preset == "centre8" else orc.PRESET_CONN4)
            x = synth.round_like(synth.activations(seed, L["wid"], n_sample, L["cin"], L["H"], L["W"]), dtype)
            w = synth.kaiming_weights(seed, L["wid"], L["cout"], L["cin"], L["ksize"])
            b = synth.bias(seed, L["wid"], L["cout"])
            prepared.append((L, k, masks, x, w, b))
        _PREPARED.clear()   # one sample at a time is kept
        _PREPARED[key] = prepared
    return _PREPARED[key]


def oracle_step(layers_k, dtype, n_sample, frac=1.0, seed=0):
    """One pass of the hot path in the CPU oracle on n_sample images.  With frac < 1 each convolution
    computes only the first ceil(frac*Cout) output channels (selection and packing always see the whole
    layer).  Returns (seconds, fraction of the full per-image multiply-adds that was computed)."""
    from oracle import rtoss_oracle as orc
    odt = {"f32": orc.DT_F32, "bf16": orc.DT_BF16, "f16": orc.DT_F16}[dtype]
    act = {"none": orc.ACT_NONE, "relu": orc.ACT_RELU, "silu": orc.ACT_SILU}
    prepared, done, full = [], 0.0, 0.0
    for (L, k, masks, x, w, b) in oracle_inputs(layers_k, dtype, n_sample, seed):
        cs = max(1, min(L["cout"], int(np.ceil(frac * L["cout"]))))
        fl = synth.layer_nnz_flops(L, 1, k)
        full += fl
        done += fl * cs / L["cout"]
        prepared.append((L, k, masks, x, w, b, cs))
    t0 = time.perf_counter()
    for (L, k, masks, x, w, b, cs) in prepared:
        if L["ksize"] == 3:
            pid = orc.select_3x3(w, masks)
            val, _, _ = orc.pack_3x3(w, masks, k, pid, odt)
            wd = orc.unpack_3x3(val, L["cout"], L["cin"], masks, k, pid)
            orc.conv3x3(x, wd[:cs], b[:cs], L["stride"], act[L["act"]], odt)
        else:
            w2 = w.reshape(L["cout"], L["cin"])
            pid = orc.select_1x1(w2, masks)
            val = orc.pack_1x1(w2, masks, k, pid, odt)
            wd = orc.unpack_1x1(val, L["cout"], L["cin"], masks, k, pid)
            orc.conv1x1(x, wd[:cs], b[:cs], L["stride"], act[L["act"]], odt)
    return time.perf_counter() - t0, done / full


def cpu_baseline_sample(layers_k, dtype, N, budget_s):
    """Time the oracle on a bounded sample: one image, a fraction of the output channels sized from a
    small calibration pass so that the timed pass takes about budget_s."""
    t_cal, f_cal = oracle_step(layers_k, dtype, 1, 1.0 / 16)
    t_image = t_cal / f_cal
    frac = min(1.0, max(1.0 / 64, budget_s / max(t_image, 1e-6)))
    n = min(N, max(1, int(budget_s / t_image))) if frac >= 1.0 else 1
    t, f = oracle_step(layers_k, dtype, n, frac)
    # a workload the oracle finishes in a second or two is passed over several times (about ten seconds in all)
    passes = 1
    if t < 5.0:
        extra = min(20, int(10.0 / max(t, 1e-3)))
        ts = [t] + [oracle_step(layers_k, dtype, n, frac)[0] for _ in range(extra)]
        t, passes = float(np.mean(ts)), len(ts)
    return n * f / t, t, f, n, passes


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    N, dtype, layers_k = workload_layers(args.workload)
    # size the per-step sample so that warmup + steps stay within about two minutes
    t_cal, f_cal = oracle_step(layers_k, dtype, 1, 1.0 / 16)
    per_step = 120.0 / max(1, args.steps + args.warmup)
    frac = min(1.0, max(1.0 / 64, f_cal * per_step / max(t_cal, 1e-6)))
    for _ in range(max(args.warmup, 0)):
        oracle_step(layers_k, dtype, 1, frac)
    res = [oracle_step(layers_k, dtype, 1, frac) for _ in range(args.steps)]
    t = float(np.mean([r[0] for r in res]))
    f = res[0][1]
    value = f / t
    cores = os.cpu_count()
    sample = ("per step: 1 image of the batch of %d, the first %.3f of every layer's output channels, "
              "whole-layer select and pack; images/s = fraction / seconds") % (N, f)
    print(json.dumps({
        "impl": "reference", "metric": "pattern-sparse conv images/sec", "value": value, "unit": "images/s",
        "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup, "ms_per_step": t * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": dtype, "data": "synthetic",
        "config": {"workload": args.workload, "batch": N, "layout": "NCHW" if args.layout == "nchw" else "NHWC", "layers": len(layers_k),
                   "l2": "not applicable (CPU oracle)", "multi_gpu": "rank 0 only", "launch": "host cores"},
        "cpu_baseline": {"value": value, "unit": "images/s", "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": "images/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }))


# --------------------------------------------------------------------------- multi-rank bookkeeping

def max_over_ranks(values, device, world):
    """Replicas only: ranks exchange nothing on the data path; the timed intervals are reduced with MAX
    so that the reported time is the slowest rank's."""
    if world <= 1:
        return [float(v) for v in values]
    import torch
    import torch.distributed as dist
    t = torch.tensor([float(v) for v in values], device=device, dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(v) for v in t]


def whole_job_value(images_per_rank, world, ms_per_step):
    """Weak scaling: every rank processes its own batch; the job's images/s is the sum."""
    return world * images_per_rank / (ms_per_step * 1e-3)


# --------------------------------------------------------------------------- GPU arm

def run_network(args):
    """Whole-network replay (convolutions + glue) as one CUDA graph: the YOLOv5s-shaped backbone + neck, or the
    RetinaNet ResNet-50-FPN-shaped network behind its 7x7 stem."""
    import torch
    from paper_2303_02191_b200 import binding as rt
    torch.cuda.set_device(0)
    ctx = rt.Context(0)
    if args.workload.startswith("retinanet"):
        from paper_2303_02191_b200.retinanet_net import GpuNet
        N = 4
        net = GpuNet(ctx, N)
        xh = synth.round_like(synth.activations(0, 1, N, 64, 200, 272), "bf16")
    else:
        from paper_2303_02191_b200.yolov5s_net import GpuNet
        N = 1 if args.workload.endswith("b1") else 16
        net = GpuNet(ctx, N)
        xh = synth.round_like(synth.activations(0, 1, N, 3, 640, 640), "bf16")
    net.set_input(xh)
    flush = torch.empty(256 * 1024 * 1024, dtype=torch.uint8, device="cuda")
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        for _ in range(max(args.warmup, 3)):
            net.run(grouped=args.group, chained=args.chain)
    torch.cuda.current_stream().wait_stream(side)
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        net.run(grouped=args.group, chained=args.chain)
    graph.replay()
    torch.cuda.synchronize()
    if ctx.rtoss_device_status() != 0:
        raise SystemExit("a device-side wait of the tensor path ran out")
    sampler = ClockSampler(physical_gpu_index(0))
    sampler.start()
    ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(args.steps)]
    for s in range(args.steps):
        flush.zero_()
        ev[s][0].record()
        graph.replay()
        ev[s][1].record()
    torch.cuda.synchronize()
    clocks = sampler.stop()
    ms = float(np.mean([a.elapsed_time(b) for a, b in ev]))
    flops = sum(synth.layer_nnz_flops(L, N, 4) for L in net.layers)
    # a convolution that adds its residual operand itself is one launch; where the library declined, two
    n_glue = sum(1 for op in net.ops if op[0] not in ("conv", "convres")) + len(getattr(net, "unfused", ()))
    print(json.dumps({
        "metric": "pattern-sparse conv images/sec", "value": N / (ms * 1e-3), "unit": "images/s", "n_gpus": 1,
        "steps": args.steps, "warmup": max(args.warmup, 3), "ms_per_step": ms, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": {"workload": args.workload, "batch": N, "layout": "NHWC", "l2": "flushed between steps (256 MB write)",
                   "launch": "one CUDA graph per step", "convs": len(net.layers), "glue_kernels": n_glue,
                   "launches_per_step": net.launches,
                   "residual_adds_inside_convs": sum(1 for op in net.ops if op[0] == "convres") - len(getattr(net, "unfused", ())),
                   "note": "chained network: every layer consumes the previous layer's output"},
        "nnz_gflops_per_s": flops / (ms * 1e-3) / 1e9, "clocks": clocks, "gpu_launches": net.launches * args.steps,
    }))
    net.close()
    ctx.close()


def measure_workload(ctx, rt, dev, name, steps, warmup, args, world, rank, full, shared=False):
    """One workload on this rank's GPU: the graph-replayed step (select + pack of every weight tensor, then every
    convolution), the cold-L2 per-launch pass for the roofline, and -- with `full` -- the end-to-end leg through the
    host-buffer entry point.  Convolutions that do not depend on one another in the network (synth.independent_sets)
    go out as one rtoss_conv_group call.  `shared`: the variant with one pattern per block of 128 filters x 16
    channels for the 3x3 layers (rtoss_select_patterns_shared); its step is the convolutions alone, selection and
    packing of the variant run once, layer by layer, outside the timed region.
    Returns a dict of raw figures (times of this rank; the caller reduces over ranks)."""
    import torch
    import torch.distributed as dist
    tdt = {"f32": torch.float32, "bf16": torch.bfloat16, "f16": torch.float16}
    N, dtype, layers_k = workload_layers(name)
    elem = 4 if dtype == "f32" else 2
    cdt = rt.DTYPE_NAMES[dtype]
    preset_of = {"centre8": rt.PRESET_CENTRE8, "conn4": rt.PRESET_CONN4}
    # activations travel NHWC (what the tensor path takes) unless NCHW is asked for (FMA path)
    layout = rt.NCHW if args.layout == "nchw" else rt.NHWC

    # ---- resident inputs (replicas: every rank holds its own batch and weights; no data-path collective)
    weights, L_state = {}, []
    for (L, k, preset) in layers_k:
        masks = rt.rtoss_pattern_preset(k, preset_of[preset])
        if L["wid"] not in weights:
            w = torch.from_numpy(synth.kaiming_weights(rank, L["wid"], L["cout"], L["cin"], L["ksize"])).to(dev)
            b = torch.from_numpy(synth.bias(rank, L["wid"], L["cout"])).to(dev)
            n_k = L["cout"] * L["cin"] if L["ksize"] == 3 else (L["cout"] * L["cin"]) // 9
            pid = torch.empty(max(n_k, 1), dtype=torch.uint8, device=dev)
            weights[L["wid"]] = dict(w=w, b=b, pid=pid, packed=None, masks=masks, k=k, ksize=L["ksize"], n_k=n_k)
        Ho, Wo = synth.out_hw(L["H"], L["W"], L["stride"])
        xh = torch.from_numpy(synth.activations(rank, len(L_state), N, L["cin"], L["H"], L["W"])).to(tdt[dtype])
        yshape = (N, L["cout"], Ho, Wo)
        if layout == rt.NHWC:
            xh = xh.permute(0, 2, 3, 1).contiguous()
            yshape = (N, Ho, Wo, L["cout"])
        st = dict(L=L, k=k, x=xh.to(dev), y=torch.empty(yshape, dtype=tdt[dtype], device=dev), Ho=Ho, Wo=Wo,
                  wt=weights[L["wid"]], path=rt.PATH_FMA)
        if full:
            st["xh"] = xh.pin_memory()
            st["yh"] = torch.empty(yshape, dtype=tdt[dtype]).pin_memory()
        L_state.append(st)
    flush = torch.empty(256 * 1024 * 1024, dtype=torch.uint8, device=dev)   # larger than the 126 MB L2

    # handles are made once, layer by layer (this allocates); every step then re-selects and re-packs ALL layers
    # with the whole-model pass: two launches, whatever the number of layers
    for wt in weights.values():
        if shared and wt["ksize"] == 3:
            ctx.rtoss_select_patterns_shared(wt["w"], wt["masks"], wt["k"], 128, 16, pid=wt["pid"])
        else:
            ctx.rtoss_select_patterns(wt["w"], wt["ksize"], wt["masks"], wt["k"], pid=wt["pid"])
        wt["packed"] = ctx.rtoss_pack(wt["w"], wt["ksize"], wt["masks"], wt["k"], wt["pid"], cdt)
    batch = ctx.rtoss_batch_create(list(weights.values()))
    any3 = any(wt["ksize"] == 3 for wt in weights.values())

    def prune_weights():
        if shared:
            return 0
        batch.rtoss_batch_select_pack()
        return 2 if any3 else 1

    def conv(st, ev=None):
        L = st["L"]
        fn = ctx.rtoss_conv3x3_pattern if L["ksize"] == 3 else ctx.rtoss_conv1x1_pattern
        if ev:
            ev[0].record()
        fn(st["wt"]["packed"], st["x"], st["y"], N, L["H"], L["W"], L["stride"], layout, rt.ACT_NAMES[L["act"]], st["wt"]["b"],
           path=st["path"])
        if ev:
            ev[1].record()

    # launch units: convolutions that are independent in the network share one grouped call
    # (and, unless --no-chain, successive tower layers share a launch whose members wait for one another: rtoss_conv_chain)
    if args.group and args.chain:
        units, afters = synth.chained_units([st["L"] for st in L_state])
    else:
        units = synth.independent_sets([st["L"] for st in L_state]) if args.group else [[i] for i in range(len(L_state))]
        afters = [None] * len(units)
    unit_launches = [1] * len(units)
    # a member that waits for another reads what that one writes, as in the network (same shape by construction)
    for u, af in zip(units, afters):
        for q, m in enumerate(af or ()):
            if m:
                src = L_state[u[m.bit_length() - 1]]
                assert src["y"].shape == L_state[u[q]]["x"].shape
                L_state[u[q]]["x"] = src["y"]

    def run_unit(u, ev=None):
        """-> kernel launches made."""
        idx = units[u]
        if len(idx) == 1:
            conv(L_state[idx[0]], ev)
            return 1
        items = []
        for i in idx:
            st = L_state[i]
            L = st["L"]
            items.append(ctx.conv_item(st["wt"]["packed"], st["x"], st["y"], N, L["H"], L["W"], L["stride"], layout,
                                       rt.ACT_NAMES[L["act"]], st["wt"]["b"], path=st["path"]))
        if ev:
            ev[0].record()
        n = ctx.rtoss_conv_chain(items, afters[u]) if afters[u] else ctx.rtoss_conv_group(items)
        if ev:
            ev[1].record()
        return n

    def step(evs=None):
        n = prune_weights()
        for u in range(len(units)):
            unit_launches[u] = run_unit(u, evs[u] if evs else None)
            n += unit_launches[u]
        return n

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    # which kernel family takes each layer: the tensor path where the call qualifies, else the FMA path
    prune_weights()
    for st in L_state:
        if args.path != "fma":
            try:
                st["path"] = rt.PATH_TENSOR
                conv(st)
            except rt.RtossError as err:
                if err.status != 3:
                    raise
                st["path"] = rt.PATH_FMA
    torch.cuda.synchronize()
    if ctx.rtoss_device_status() != 0:
        raise SystemExit("a device-side wait of the tensor path ran out")
    for _ in range(max(warmup, 3)):
        step()
        flush.zero_()
    barrier()
    if ctx.rtoss_device_status() != 0:
        # A launch whose members wait for one another needs all its CTAs on the device together; if something else holds
        # SMs the bounded wait runs out.  Then the dependent convolutions get launches of their own, as without --chain.
        if not any(a is not None for a in afters):
            raise SystemExit("a device-side wait of the tensor path ran out")
        sys.stderr.write("a wait inside a shared launch ran out: dependent convolutions get launches of their own\n")
        units[:] = synth.independent_sets([st["L"] for st in L_state])
        afters[:] = [None] * len(units)
        unit_launches[:] = [1] * len(units)
        for _ in range(max(warmup, 3)):
            step()
            flush.zero_()
        barrier()
        if ctx.rtoss_device_status() != 0:
            raise SystemExit("a device-side wait of the tensor path ran out")

    # The step is launch-bound when driven call by call from Python, so the timed region replays it as ONE CUDA
    # graph, as a deployment would.
    graph = None
    launches_per_step = 0
    if args.graph:
        try:
            side = torch.cuda.Stream()
            side.wait_stream(torch.cuda.current_stream())
            with torch.cuda.stream(side):
                step()
            torch.cuda.current_stream().wait_stream(side)
            torch.cuda.synchronize()
            graph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(graph):
                launches_per_step = step()
            graph.replay()
            torch.cuda.synchronize()
        except Exception as err:  # keep measuring, say so in the line
            sys.stderr.write("graph capture failed, timing eager launches: %r\n" % (err,))
            graph = None
            torch.cuda.synchronize()
    sampler = ClockSampler(physical_gpu_index(int(os.environ.get("LOCAL_RANK", "0"))))
    sampler.start()
    step_ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(steps)]
    launches = 0
    barrier()
    for s in range(steps):
        flush.zero_()                       # L2 flush between timed iterations, outside the step's events
        step_ev[s][0].record()
        if graph is not None:
            graph.replay()
            launches += launches_per_step
        else:
            launches += step()
        step_ev[s][1].record()
    barrier()
    total_ms = float(np.array([a.elapsed_time(b) for a, b in step_ev]).sum())

    # Per-launch durations for the roofline: the same K steps again, the whole-model select + pack and every
    # convolution each between its own pair of events right after a 256 MB flush write (cold L2).  The pass is
    # captured once into a CUDA graph whose event records are graph nodes (external events) and replayed K times,
    # so the host's enqueue time cannot leak into an interval; if the capture is not available the launches are
    # issued one by one (the flush write queued before each launch then keeps the GPU busy while the host enqueues).
    conv_ms, prune_ms = None, None
    if args.graph:
        try:
            gev = [(torch.cuda.Event(enable_timing=True, external=True), torch.cuda.Event(enable_timing=True, external=True))
                   for _ in range(len(units) + 1)]
            kgraph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(kgraph):
                flush.zero_()
                gev[-1][0].record()
                prune_weights()
                gev[-1][1].record()
                for u in range(len(units)):
                    flush.zero_()
                    run_unit(u, gev[u])
            acc = np.zeros(len(units) + 1)
            for s in range(steps):
                kgraph.replay()
                torch.cuda.synchronize()
                acc += np.array([a.elapsed_time(b) for a, b in gev])
            conv_ms, prune_ms = acc[:-1] / steps, float(acc[-1] / steps)
        except Exception as err:
            sys.stderr.write("per-kernel timing graph not available, timing eager launches: %r\n" % (err,))
            torch.cuda.synchronize()
            conv_ms = None
    if conv_ms is None:
        conv_ev = [[(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(len(units) + 1)]
                   for _ in range(steps)]
        for s in range(steps):
            flush.zero_()
            conv_ev[s][-1][0].record()
            prune_weights()
            conv_ev[s][-1][1].record()
            for u in range(len(units)):
                flush.zero_()
                run_unit(u, conv_ev[s][u])
        barrier()
        allms = np.array([[a.elapsed_time(b) for a, b in row] for row in conv_ev]).mean(axis=0)
        conv_ms, prune_ms = allms[:-1], float(allms[-1])
    barrier()
    clocks = sampler.stop()
    if ctx.rtoss_device_status() != 0:
        raise SystemExit("a device-side wait of the tensor path ran out during the timed region")

    res = dict(name=name, N=N, dtype=dtype, elem=elem, layout="NHWC" if layout == rt.NHWC else "NCHW", total_ms=total_ms,
               steps=steps, launches=launches, graph=graph is not None, conv_ms=conv_ms, prune_ms=prune_ms, clocks=clocks,
               units=units, unit_launches=list(unit_launches), shared=shared,
               layers=[st["L"] for st in L_state], ks=[st["k"] for st in L_state],
               on_tc=[st["path"] == rt.PATH_TENSOR for st in L_state],
               weights=[dict(n_k=wt["n_k"], k=wt["k"], ksize=wt["ksize"]) for wt in weights.values()], e2e_s=None)

    # ---- end to end through the host-buffer entry point (pinned host tensors, copies inside the timed region)
    if full:
        torch.cuda.synchronize()
        res["h2d"] = sum(st["xh"].numel() * elem for st in L_state)
        res["d2h"] = sum(st["yh"].numel() * elem for st in L_state)
        e2e_steps = max(2, min(steps, 20, int(2e10 / (res["h2d"] + res["d2h"]))))   # bounded: about 20 GB over PCIe at most
        for st in L_state[:1]:
            ctx.rtoss_conv_pattern_host(st["wt"]["packed"], st["xh"], st["yh"], N, st["L"]["H"], st["L"]["W"], st["L"]["stride"],
                                        layout, rt.ACT_NAMES[st["L"]["act"]], st["wt"]["b"], path=st["path"])
        barrier()
        t0 = time.perf_counter()
        for _ in range(e2e_steps):
            prune_weights()
            torch.cuda.synchronize()   # the host-buffer call runs on the context's own streams: packing must be complete
            for st in L_state:
                L = st["L"]
                ctx.rtoss_conv_pattern_host(st["wt"]["packed"], st["xh"], st["yh"], N, L["H"], L["W"], L["stride"], layout,
                                            rt.ACT_NAMES[L["act"]], st["wt"]["b"], path=st["path"])
        torch.cuda.synchronize()
        res["e2e_s"] = (time.perf_counter() - t0) / e2e_steps

    torch.cuda.synchronize()
    batch.close()
    for wt in weights.values():
        if wt["packed"] is not None:
            wt["packed"].close()
    del L_state, weights, flush
    torch.cuda.empty_cache()
    return res


def roofline_of(res, hbm_peak, tc_peak, peak_kind):
    """Roofline figures of one measured workload.  Per launch: T_roof = max(algorithmic bytes / HBM copy peak,
    non-zero FLOP / peak of the pipe the kernel uses); the stack's fraction is sum(T_roof) / sum(T_measured) over the
    cold-L2 per-launch pass; the dominant kernel (largest share of that pass) gets its own record."""
    N, elem = res["N"], res["elem"]
    flops = np.array([synth.layer_nnz_flops(L, N, k) for L, k in zip(res["layers"], res["ks"])])
    bytes_ = np.array([synth.layer_bytes(L, N, k, elem) for L, k in zip(res["layers"], res["ks"])], dtype=np.float64)
    # pipe peak per layer: the measured bf16 tensor peak; fp32 on the tensor path issues tf32 instructions (half the bf16
    # rate) three times per product (head x head, head x remainder, remainder x head); else the nominal FMA peak
    tc_eff = tc_peak if res["dtype"] != "f32" else tc_peak / 6
    pipe = np.array([tc_eff if tc else ALU_PEAK_TFLOPS for tc in res["on_tc"]]) * 1e12
    t_pipe, t_hbm = flops / pipe, bytes_ / (hbm_peak * 1e9)
    t_roof = np.maximum(t_pipe, t_hbm)
    t_meas = res["conv_ms"] * 1e-3          # one entry per launch unit (a unit of several layers is one grouped call)
    units = res["units"]
    u_roof = np.array([t_roof[u].sum() for u in units])
    u_flops = np.array([flops[u].sum() for u in units])
    u_bytes = np.array([bytes_[u].sum() for u in units])
    stack_frac = float(t_roof.sum() / t_meas.sum())
    # the dominant kernel: units of one composition (the shapes of their layers) share a kernel configuration; the
    # composition with the largest share of the cold pass
    shape_of = lambda L: (L["ksize"], L["stride"], L["cin"], L["cout"], L["H"], L["W"])
    share = {}
    for ui, u in enumerate(units):
        share.setdefault(tuple(shape_of(res["layers"][i]) for i in u), []).append(ui)
    top_shape = max(share, key=lambda sh: t_meas[share[sh]].sum())
    idx = share[top_shape]
    top = idx[int(np.argmax(t_meas[idx]))]
    members = units[top]
    on_tc = res["on_tc"][members[0]]
    t_top = float(np.mean(t_meas[idx]))
    if t_pipe[members].sum() >= t_hbm[members].sum():
        dom = {"bound": ("tensor (tf32 x3)" if res["dtype"] == "f32" else "tensor") if on_tc else "alu",
               "achieved": u_flops[top] / t_top / 1e12, "peak": pipe[members[0]] / 1e12, "unit": "TFLOP/s",
               "peak_kind": ("of %s (bf16 cuBLAS, sustained)%s" % (peak_kind, " / 2 (tf32) / 3 (products per tap)" if res["dtype"] == "f32" else "")) if on_tc
               else "nominal, not measured: 148 SM x 128 FMA lanes x 2 x 1.965 GHz"}
    else:
        dom = {"bound": "hbm", "achieved": u_bytes[top] / t_top / 1e9, "peak": hbm_peak, "unit": "GB/s", "peak_kind": "of " + peak_kind}
    dom["frac"] = float(u_roof[top] / t_top)   # sum of the members' roofline times / the launch's time
    L = res["layers"][members[0]]
    dom["kernel"] = ("conv_tc_kernel " if on_tc else "conv_alu_kernel ") + L["name"] + " k=%d" % res["ks"][members[0]] + \
                    ("" if len(members) == 1 else " + %d more convolutions in the same launch" % (len(members) - 1))
    dom["convolutions_per_launch"] = len(members)
    dom["launches_of_this_kind"] = len(idx)
    dom["share_of_cold_pass"] = float(t_meas[idx].sum() / t_meas.sum())
    dom["kernel_ms"] = t_top * 1e3
    dom["nnz_flop_per_launch"] = float(u_flops[top])
    dom["algorithmic_bytes_per_launch"] = float(u_bytes[top])
    dom["traffic"] = ncu_traffic(res["name"], L["name"] + ("+%d" % (len(members) - 1) if len(members) > 1 else ""), res["ks"][members[0]])
    # whole-model selection + packing: 36 B read per kernel (nine fp32 weights), k values + the id + the order entry written
    sp_bytes = float(sum(w["n_k"] * (36 + w["k"] * elem + (5 if w["ksize"] == 3 else 1)) for w in res["weights"]))
    sp = {"kernels": int(sum(w["n_k"] for w in res["weights"])), "launches": 2 if any(w["ksize"] == 3 for w in res["weights"]) else 1,
          "algorithmic_bytes": sp_bytes, "us": res["prune_ms"] * 1e3, "bound": "hbm",
          "achieved_gbs": sp_bytes / (res["prune_ms"] * 1e-3) / 1e9, "peak_gbs": hbm_peak,
          "frac": sp_bytes / (res["prune_ms"] * 1e-3) / 1e9 / hbm_peak,
          "note": "cold L2; besides the algorithmic bytes the pass writes the tensor path's 9-tap weight expansion"}
    tensor_share = float(t_roof[t_pipe >= t_hbm].sum() / t_roof.sum())
    return dict(stack_frac=stack_frac, sum_roof_ms=float(t_roof.sum() * 1e3), sum_cold_ms=float(t_meas.sum() * 1e3),
                tensor_share=tensor_share, dominant=dom, select_pack=sp, flops=flops, bytes=bytes_, t_roof=t_roof,
                t_pipe=t_pipe, t_hbm=t_hbm, u_roof=u_roof)


OTHER_WORKLOADS = ("layer32", "layer128", "yolov5s_b1", "yolov5s_b16")


def run_gpu(args):
    import torch
    import torch.distributed as dist
    from paper_2303_02191_b200 import binding as rt

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the hot path has no CPU fallback")
    torch.cuda.set_device(local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    dev = torch.device("cuda", local_rank)
    ctx = rt.Context(local_rank)

    res = measure_workload(ctx, rt, dev, args.workload, args.steps, args.warmup, args, world, rank, full=True)
    total_ms, e2e_s = max_over_ranks([res["total_ms"], res["e2e_s"]], dev, world)
    others, variant = {}, None
    if args.others and world == 1:
        for name in OTHER_WORKLOADS:
            if name != args.workload:
                others[name] = measure_workload(ctx, rt, dev, name, min(args.steps, 20), 3, args, 1, rank, full=False)
        if res["dtype"] != "f32":
            variant = measure_workload(ctx, rt, dev, args.workload, min(args.steps, 20), 3, args, 1, rank, full=False, shared=True)

    if rank == 0:
        N, dtype = res["N"], res["dtype"]
        ms_per_step = total_ms / args.steps
        value = whole_job_value(N, world, ms_per_step)
        hbm_peak, tc_peak, peak_kind = read_peaks()
        rf = roofline_of(res, hbm_peak, tc_peak, peak_kind)
        dom = rf["dominant"]
        tensor_led = rf["tensor_share"] >= 0.5
        roof = {
            "bound": "tensor" if tensor_led else "hbm",
            "frac": rf["stack_frac"],
            # the stack's fraction expressed in the unit of the bound that holds most of the roofline time
            "achieved": rf["stack_frac"] * (tc_peak if tensor_led else hbm_peak), "peak": tc_peak if tensor_led else hbm_peak,
            "unit": "TFLOP/s" if tensor_led else "GB/s",
            "peak_kind": "of %s (%s)" % (peak_kind, "bf16 cuBLAS, sustained" if tensor_led else "copy"),
            "traffic": dom.pop("traffic"),
            "definition": "stack figure: sum over launches of max(algorithmic bytes / HBM copy peak, non-zero FLOP / pipe peak) "
                          "divided by the sum of the cold-L2 CUDA-event times of the same launches; 'achieved' = frac x peak; "
                          "share of the roofline time that is tensor-bound: %.2f" % rf["tensor_share"],
            "sum_roofline_ms": rf["sum_roof_ms"], "sum_cold_kernel_ms": rf["sum_cold_ms"],
            # the same roofline time (convolutions + the select/pack pass at the copy peak) against the graph-replayed step,
            # where a launch's latency and prologue overlap the kernel before it; the cold pass pays them once per launch
            "frac_in_step": (rf["sum_roof_ms"] + rf["select_pack"]["algorithmic_bytes"] / (hbm_peak * 1e9) * 1e3) / ms_per_step,
            "dominant_kernel": dom, "select_pack": rf["select_pack"],
            "notes": ["both convolution paths multiply the pruned taps as zeros: a tensor-bound layer cannot exceed k/9 of its "
                      "non-zero roofline",
                      "the tensor path reads the 9-tap dense expansion of the weights (9/k x the packed bytes the roofline counts)",
                      "the FMA-pipe peak is the nominal 148 x 128 x 2 x 1.965 GHz, not a measured one"],
        }
        out = {
            "metric": "pattern-sparse conv images/sec", "value": value, "unit": "images/s", "n_gpus": world,
            "steps": args.steps, "warmup": max(args.warmup, 3), "ms_per_step": ms_per_step, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": dtype, "data": "synthetic",
            "config": {"workload": args.workload, "batch": N, "layout": res["layout"], "layers": len(res["layers"]),
                       "l2": "flushed between steps (256 MB write)", "multi_gpu": "replicas only",
                       "launch": "one CUDA graph per step" if res["graph"] else "eager",
                       "grouping": ("independent convolutions%s share a launch: %d launches for %d convolutions"
                                    % (" and successive tower layers" if args.chain else "", sum(res["unit_launches"]), len(res["layers"])))
                                   if args.group else "one launch per convolution"},
            "paths": {"tensor_path_layers": int(sum(res["on_tc"])), "fma_path_layers": int(len(res["on_tc"]) - sum(res["on_tc"]))},
            "nnz_gflops_per_s": float(rf["flops"].sum()) / (ms_per_step * 1e-3) / 1e9 * world,
            "conv_ms": [float(v) for v in res["conv_ms"]] if len(res["conv_ms"]) <= 8 else None,
            "conv_ms_sum": float(res["conv_ms"].sum()),
            "roofline": roof, "clocks": res["clocks"],
            "e2e": {"value": world * N / e2e_s, "unit": "images/s", "h2d_bytes_per_step": res["h2d"], "d2h_bytes_per_step": res["d2h"]},
            "gpu_launches": res["launches"],
        }
        if others:
            out["others"] = {}
            for name, r in others.items():
                orf = roofline_of(r, hbm_peak, tc_peak, peak_kind)
                ms = r["total_ms"] / r["steps"]
                d = orf["dominant"]
                out["others"][name] = {
                    "batch": r["N"], "dtype": r["dtype"], "steps": r["steps"], "ms_per_step": ms, "images_per_s": r["N"] / (ms * 1e-3),
                    "nnz_gflops_per_s": float(orf["flops"].sum()) / (ms * 1e-3) / 1e9, "roofline_frac": orf["stack_frac"],
                    "sum_roofline_ms": orf["sum_roof_ms"], "sum_cold_kernel_ms": orf["sum_cold_ms"],
                    "dominant_kernel": {"kernel": d["kernel"], "bound": d["bound"], "frac": d["frac"], "kernel_ms": d["kernel_ms"]},
                    "select_pack_us": orf["select_pack"]["us"], "select_pack_frac": orf["select_pack"]["frac"],
                    "tensor_path_layers": int(sum(r["on_tc"])), "fma_path_layers": int(len(r["on_tc"]) - sum(r["on_tc"])),
                    "clocks": r["clocks"], "gpu_launches": r["launches"]}
        if variant is not None:
            vrf = roofline_of(variant, hbm_peak, tc_peak, peak_kind)
            vms = variant["total_ms"] / variant["steps"]
            vd = vrf["dominant"]
            out["shared_pattern_variant"] = {
                "what": "the 3x3 layers pruned with ONE pattern per block of 128 filters x 16 input channels "
                        "(rtoss_select_patterns_shared) instead of one per kernel: a different, coarser pruning result (its "
                        "effect on detection accuracy is not measured here); the tensor path then issues only the k kept taps",
                "step": "the convolutions only (selection and packing of the variant run once, outside the timed region)",
                "steps": variant["steps"], "ms_per_step": vms, "images_per_s": variant["N"] / (vms * 1e-3),
                "nnz_gflops_per_s": float(vrf["flops"].sum()) / (vms * 1e-3) / 1e9,
                "roofline_frac": vrf["stack_frac"], "sum_roofline_ms": vrf["sum_roof_ms"], "sum_cold_kernel_ms": vrf["sum_cold_ms"],
                "dominant_kernel": {k_: vd[k_] for k_ in ("kernel", "bound", "achieved", "peak", "unit", "frac", "kernel_ms",
                                                          "convolutions_per_launch", "share_of_cold_pass")},
                "clocks": variant["clocks"], "gpu_launches": variant["launches"]}
        if args.layers_csv:
            # per-layer table: cold-L2 kernel time next to the two roofline terms at non-zero FLOPs
            with open(args.layers_csv, "w") as f:
                f.write("launch,convolutions,launches,ksize,cin,cout,H,W,stride,k,path,kernel_us,hbm_us,pipe_us,roofline_us,frac\n")
                for ui, u in enumerate(res["units"]):
                    L, k, tc = res["layers"][u[0]], res["ks"][u[0]], res["on_tc"][u[0]]
                    ms = res["conv_ms"][ui]
                    f.write("%s,%d,%d,%d,%d,%d,%d,%d,%d,%d,%s,%.2f,%.2f,%.2f,%.2f,%.3f\n" % (
                        L["name"], len(u), res["unit_launches"][ui], L["ksize"], L["cin"], L["cout"], L["H"], L["W"], L["stride"], k,
                        "tensor" if tc else "fma", ms * 1e3, rf["t_hbm"][u].sum() * 1e6, rf["t_pipe"][u].sum() * 1e6,
                        rf["u_roof"][ui] * 1e6, rf["u_roof"][ui] * 1e3 / ms))
        if args.cpu_baseline:
            _, _, layers_k = workload_layers(args.workload)
            v_cpu, t_cpu, f_cpu, n_cpu, p_cpu = cpu_baseline_sample(layers_k, dtype, N, 15.0)
            out["cpu_baseline"] = {"value": v_cpu, "unit": "images/s", "cores": os.cpu_count(), "kind": "oracle",
                                   "sample": "%d image(s) of the batch of %d, the first %.3f of every layer's output channels, "
                                             "%d pass(es) of %.1f s each (mean); images/s = images x fraction / seconds"
                                             % (n_cpu, N, f_cpu, p_cpu, t_cpu)}
        print(json.dumps(out))
    torch.cuda.synchronize()
    ctx.close()
    if world > 1:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=30)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="retinanet_b4")
    ap.add_argument("--no-chain", dest="chain", action="store_false",
                    help="dependent convolutions do not share launches (rtoss_conv_chain is not used)")
    ap.add_argument("--no-others", dest="others", action="store_false",
                    help="skip the sub-records of the other configurations (layer32, layer128, yolov5s_b1, yolov5s_b16)")
    ap.add_argument("--no-cpu-baseline", dest="cpu_baseline", action="store_false")
    ap.add_argument("--no-graph", dest="graph", action="store_false", help="time eager launches instead of a CUDA graph")
    ap.add_argument("--no-group", dest="group", action="store_false", help="one launch per convolution (no rtoss_conv_group)")
    ap.add_argument("--path", default="auto", choices=["auto", "fma"], help="fma: keep every layer on the FMA path")
    ap.add_argument("--layers-csv", default=None, help="write the per-layer kernel times and roofline terms to this file")
    ap.add_argument("--layout", default="auto", choices=["auto", "nchw"], help="nchw: NCHW activations also for 16-bit types")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
        return
    if args.workload in ("yolov5s_net_b1", "yolov5s_net_b16", "retinanet_net_b4"):
        run_network(args)
        return
    if int(os.environ.get("WORLD_SIZE", "1")) > 1 or args.gpus == 1:
        if int(os.environ.get("WORLD_SIZE", "1")) > 1:
            args.cpu_baseline = False
        run_gpu(args)
    else:
        raise SystemExit("for --gpus N > 1 launch with: python -m torch.distributed.run --nproc-per-node N bench.py --gpus N")


if __name__ == "__main__":
    main()
