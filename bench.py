#!/usr/bin/env python
"""Benchmark of the R-TOSS hot path on B200.

A step is one pass of the whole hot path over one batch of synthetic input:
pattern selection (Algorithm 2 / 3 of arXiv 2303.02191), packing, and the
pattern-sparse convolution, for each layer of the workload.  Default workload
"layer128": batch 8, bf16 --
  3x3 128->128 @80x80 with 3-entry patterns, the same layer with 2-entry
  patterns, and a 1x1 256->128 @80x80 whose weights are regrouped into 3x3
  blocks and pruned with the 3-entry patterns.
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
    raise SystemExit("unknown workload " + name)


# DRAM bytes per launch (dram__bytes_read.sum + dram__bytes_write.sum) of a workload's dominant kernel from one
# ncu capture (caches flushed before every pass; the commands are in profiles/conv_tc_layer128.md), valid
# for the kernel source whose hash is recorded with it: once conv_tc.cu changes the figure is withheld (null).
# 13.5 MB = the activations and the weights once; the 13.1 MB of outputs are still dirty in the 126 MB L2 when the
# kernel ends, so the capture sees no write.
NCU_TRAFFIC = {("layer128", "conv3x3_128", 3): (13506304, "1977b3266a0d51c6")}


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

def oracle_step(layers_k, dtype, n_sample, frac=1.0, seed=0):
    """One pass of the hot path in the CPU oracle on n_sample images.  With frac < 1 each convolution
    computes only the first ceil(frac*Cout) output channels (selection and packing always see the whole
    layer).  Returns (seconds, fraction of the full per-image multiply-adds that was computed)."""
    from oracle import rtoss_oracle as orc
    odt = {"f32": orc.DT_F32, "bf16": orc.DT_BF16, "f16": orc.DT_F16}[dtype]
    act = {"none": orc.ACT_NONE, "relu": orc.ACT_RELU, "silu": orc.ACT_SILU}
    prepared, done, full = [], 0.0, 0.0
    for (L, k, preset) in layers_k:
        masks = orc.pattern_preset(k, orc.PRESET_CENTRE8 if preset == "centre8" else orc.PRESET_CONN4)
        x = synth.round_like(synth.activations(seed, L["wid"], n_sample, L["cin"], L["H"], L["W"]), dtype)
        w = synth.kaiming_weights(seed, L["wid"], L["cout"], L["cin"], L["ksize"])
        b = synth.bias(seed, L["wid"], L["cout"])
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
        "config": {"workload": args.workload, "batch": N},
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
            net.run()
    torch.cuda.current_stream().wait_stream(side)
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        net.run()
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
                   "residual_adds_inside_convs": sum(1 for op in net.ops if op[0] == "convres") - len(getattr(net, "unfused", ())),
                   "note": "chained network: every layer consumes the previous layer's output"},
        "nnz_gflops_per_s": flops / (ms * 1e-3) / 1e9, "clocks": clocks, "gpu_launches": (len(net.layers) + n_glue) * args.steps,
    }))
    net.close()
    ctx.close()


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
    tdt = {"f32": torch.float32, "bf16": torch.bfloat16, "f16": torch.float16}

    N, dtype, layers_k = workload_layers(args.workload)
    elem = 4 if dtype == "f32" else 2
    cdt = rt.DTYPE_NAMES[dtype]
    preset_of = {"centre8": rt.PRESET_CENTRE8, "conn4": rt.PRESET_CONN4}
    # 16-bit activations travel NHWC (what the tensor path takes), fp32 NCHW
    layout = rt.NCHW if (dtype == "f32" or args.layout == "nchw") else rt.NHWC

    # ---- resident inputs (replicas: every rank holds its own batch and weights; no data-path collective)
    weights, L_state = {}, []
    for (L, k, preset) in layers_k:
        masks = rt.rtoss_pattern_preset(k, preset_of[preset])
        if L["wid"] not in weights:
            w = torch.from_numpy(synth.kaiming_weights(rank, L["wid"], L["cout"], L["cin"], L["ksize"])).to(dev)
            b = torch.from_numpy(synth.bias(rank, L["wid"], L["cout"])).to(dev)
            n_k = L["cout"] * L["cin"] if L["ksize"] == 3 else (L["cout"] * L["cin"]) // 9
            pid = torch.empty(max(n_k, 1), dtype=torch.uint8, device=dev)
            weights[L["wid"]] = dict(w=w, b=b, pid=pid, packed=None, masks=masks, k=k, ksize=L["ksize"])
        Ho, Wo = synth.out_hw(L["H"], L["W"], L["stride"])
        xh = torch.from_numpy(synth.activations(rank, len(L_state), N, L["cin"], L["H"], L["W"])).to(tdt[dtype])
        yshape = (N, L["cout"], Ho, Wo)
        if layout == rt.NHWC:
            xh = xh.permute(0, 2, 3, 1).contiguous()
            yshape = (N, Ho, Wo, L["cout"])
        st = dict(L=L, k=k, x=xh.to(dev), y=torch.empty(yshape, dtype=tdt[dtype], device=dev),
                  xh=xh.pin_memory(), yh=torch.empty(yshape, dtype=tdt[dtype]).pin_memory(),
                  Ho=Ho, Wo=Wo, wt=weights[L["wid"]], path=rt.PATH_FMA)
        L_state.append(st)
    flush = torch.empty(256 * 1024 * 1024, dtype=torch.uint8, device=dev)   # larger than the 126 MB L2

    # handles are made once, layer by layer (this allocates); every step then re-selects and re-packs ALL layers
    # with the whole-model pass: two launches, whatever the number of layers
    for wt in weights.values():
        ctx.rtoss_select_patterns(wt["w"], wt["ksize"], wt["masks"], wt["k"], pid=wt["pid"])
        wt["packed"] = ctx.rtoss_pack(wt["w"], wt["ksize"], wt["masks"], wt["k"], wt["pid"], cdt)
    batch = ctx.rtoss_batch_create(list(weights.values()))
    any3 = any(wt["ksize"] == 3 for wt in weights.values())

    def prune_weights():
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

    def step(evs=None):
        n = prune_weights()
        for i, st in enumerate(L_state):
            conv(st, evs[i] if evs else None)
        return n + len(L_state)

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
    for _ in range(max(args.warmup, 3)):
        step()
        flush.zero_()
    barrier()

    # The step is launch-bound when driven call by call from Python (about twenty small launches for
    # ~100 us of GPU work), so the timed region replays it as ONE CUDA graph, as a deployment would.
    graph = None
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
    sampler = ClockSampler(physical_gpu_index(local_rank))
    sampler.start()
    step_ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(args.steps)]
    launches = 0
    barrier()
    for s in range(args.steps):
        flush.zero_()                       # L2 flush between timed iterations, outside the step's events
        step_ev[s][0].record()
        if graph is not None:
            graph.replay()
            launches += launches_per_step
        else:
            launches += step()
        step_ev[s][1].record()
    barrier()
    step_ms = np.array([a.elapsed_time(b) for a, b in step_ev])
    total_ms = float(step_ms.sum())

    # Per-kernel durations for the roofline: the same K steps again, every convolution between its own pair of
    # events right after a 256 MB flush write (cold L2).  The pass is captured once into a CUDA graph whose event
    # records are graph nodes (external events) and replayed K times, so the host's enqueue time cannot leak into
    # an interval; if the capture is not available the launches are issued one by one (the flush write queued
    # before each launch then keeps the GPU busy while the host enqueues it).
    conv_ms = None
    if args.graph:
        try:
            gev = [(torch.cuda.Event(enable_timing=True, external=True), torch.cuda.Event(enable_timing=True, external=True))
                   for _ in L_state]
            kgraph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(kgraph):
                prune_weights()
                for i, st in enumerate(L_state):
                    flush.zero_()
                    conv(st, gev[i])
            acc = np.zeros(len(L_state))
            for s in range(args.steps):
                kgraph.replay()
                torch.cuda.synchronize()
                acc += np.array([a.elapsed_time(b) for a, b in gev])
            conv_ms = acc / args.steps
        except Exception as err:
            sys.stderr.write("per-kernel timing graph not available, timing eager launches: %r\n" % (err,))
            torch.cuda.synchronize()
            conv_ms = None
    if conv_ms is None:
        conv_ev = [[(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in L_state]
                   for _ in range(args.steps)]
        for s in range(args.steps):
            prune_weights()
            for i, st in enumerate(L_state):
                flush.zero_()
                conv(st, conv_ev[s][i])
        barrier()
        conv_ms = np.array([[a.elapsed_time(b) for a, b in row] for row in conv_ev]).mean(axis=0)
    barrier()
    clocks = sampler.stop()

    # ---- end to end through the host-buffer entry point (pinned host tensors, copies inside the timed region)
    torch.cuda.synchronize()
    h2d = sum(st["xh"].numel() * elem for st in L_state)
    d2h = sum(st["yh"].numel() * elem for st in L_state)
    e2e_steps = max(2, min(args.steps, 20, int(2e10 / (h2d + d2h))))   # bounded: about 20 GB over PCIe at most
    for st in L_state[:1]:
        ctx.rtoss_conv_pattern_host(st["wt"]["packed"], st["xh"], st["yh"], N, st["L"]["H"], st["L"]["W"], st["L"]["stride"],
                                    layout, rt.ACT_NAMES[st["L"]["act"]], st["wt"]["b"], path=st["path"])
    barrier()
    t0 = time.perf_counter()
    for _ in range(e2e_steps):
        prune_weights()
        torch.cuda.synchronize()
        for st in L_state:
            L = st["L"]
            ctx.rtoss_conv_pattern_host(st["wt"]["packed"], st["xh"], st["yh"], N, L["H"], L["W"], L["stride"], layout,
                                        rt.ACT_NAMES[L["act"]], st["wt"]["b"], path=st["path"])
    torch.cuda.synchronize()
    e2e_s = (time.perf_counter() - t0) / e2e_steps

    total_ms, e2e_s = max_over_ranks([total_ms, e2e_s], dev, world)

    if rank == 0:
        ms_per_step = total_ms / args.steps
        value = whole_job_value(N, world, ms_per_step)
        flops = [synth.layer_nnz_flops(st["L"], N, st["k"]) for st in L_state]
        bytes_ = [synth.layer_bytes(st["L"], N, st["k"], elem) for st in L_state]
        top = int(np.argmax(conv_ms))
        hbm_peak, tc_peak, peak_kind = read_peaks()
        t_top = conv_ms[top] * 1e-3
        on_tc = L_state[top]["path"] == rt.PATH_TENSOR
        pipe_peak = tc_peak if on_tc else ALU_PEAK_TFLOPS          # TFLOP/s of the pipe the kernel uses
        pipe_t, hbm_t = flops[top] / (pipe_peak * 1e12), bytes_[top] / (hbm_peak * 1e9)
        if pipe_t >= hbm_t:
            roof = {"bound": "tensor" if on_tc else "alu", "achieved": flops[top] / t_top / 1e12, "peak": pipe_peak,
                    "unit": "TFLOP/s",
                    "peak_kind": ("of %s (bf16 cuBLAS, sustained)" % peak_kind) if on_tc
                    else "derived: 148 SM x 128 FMA lanes x 2 x 1.965 GHz"}
        else:
            roof = {"bound": "hbm", "achieved": bytes_[top] / t_top / 1e9, "peak": hbm_peak, "unit": "GB/s",
                    "peak_kind": "of " + peak_kind}
        roof["frac"] = roof["achieved"] / roof["peak"]
        roof["traffic"] = ncu_traffic(args.workload, L_state[top]["L"]["name"], L_state[top]["k"])
        roof["kernel"] = ("conv_tc_kernel " if on_tc else "conv_alu_kernel ") + L_state[top]["L"]["name"] + " k=%d" % L_state[top]["k"]
        roof["kernel_ms"] = float(conv_ms[top])
        roof["nnz_flop_per_launch"] = flops[top]
        roof["algorithmic_bytes_per_launch"] = bytes_[top]
        out = {
            "metric": "pattern-sparse conv images/sec", "value": value, "unit": "images/s", "n_gpus": world,
            "steps": args.steps, "warmup": max(args.warmup, 3), "ms_per_step": ms_per_step, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": dtype, "data": "synthetic",
            "config": {"workload": args.workload, "batch": N, "layout": "NHWC" if layout == rt.NHWC else "NCHW",
                       "l2": "flushed between steps (256 MB write)", "layers": len(L_state), "multi_gpu": "replicas only",
                       "launch": "one CUDA graph per step" if graph is not None else "eager",
                       "tensor_path_layers": sum(1 for st in L_state if st["path"] == rt.PATH_TENSOR),
                       "fma_path_layers": sum(1 for st in L_state if st["path"] == rt.PATH_FMA)},
            "nnz_gflops_per_s": sum(flops) / (ms_per_step * 1e-3) / 1e9 * world,
            "conv_ms": [float(v) for v in conv_ms] if len(conv_ms) <= 8 else None,
            "conv_ms_sum": float(conv_ms.sum()),
            "roofline": roof, "clocks": clocks,
            "e2e": {"value": world * N / e2e_s, "unit": "images/s", "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h},
            "gpu_launches": launches,
        }
        if args.layers_csv:
            # per-layer table: cold-L2 kernel time next to the two roofline terms at non-zero FLOPs
            with open(args.layers_csv, "w") as f:
                f.write("layer,ksize,cin,cout,H,W,stride,k,path,kernel_us,hbm_us,pipe_us,frac\n")
                for st, ms, fl, by in zip(L_state, conv_ms, flops, bytes_):
                    L = st["L"]
                    tc = st["path"] == rt.PATH_TENSOR
                    pipe_us = fl / ((tc_peak if tc else ALU_PEAK_TFLOPS) * 1e12) * 1e6
                    hbm_us = by / (hbm_peak * 1e9) * 1e6
                    f.write("%s,%d,%d,%d,%d,%d,%d,%d,%s,%.2f,%.2f,%.2f,%.3f\n" % (
                        L["name"], L["ksize"], L["cin"], L["cout"], L["H"], L["W"], L["stride"], st["k"],
                        "tensor" if tc else "fma", ms * 1e3, hbm_us, pipe_us, max(hbm_us, pipe_us) / (ms * 1e3)))
        if args.cpu_baseline:
            v_cpu, t_cpu, f_cpu, n_cpu, p_cpu = cpu_baseline_sample(layers_k, dtype, N, 15.0)
            out["cpu_baseline"] = {"value": v_cpu, "unit": "images/s", "cores": os.cpu_count(), "kind": "oracle",
                                   "sample": "%d image(s) of the batch of %d, the first %.3f of every layer's output channels, "
                                             "%d pass(es) of %.1f s each (mean); images/s = images x fraction / seconds"
                                             % (n_cpu, N, f_cpu, p_cpu, t_cpu)}
        print(json.dumps(out))
    torch.cuda.synchronize()
    batch.close()
    for wt in weights.values():
        if wt["packed"] is not None:
            wt["packed"].close()
    ctx.close()
    if world > 1:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="layer128")
    ap.add_argument("--no-cpu-baseline", dest="cpu_baseline", action="store_false")
    ap.add_argument("--no-graph", dest="graph", action="store_false", help="time eager launches instead of a CUDA graph")
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
