"""Sweep of isolated 3x3 pattern convolutions (stride 1, pad 1):
Cin = Cout in {64, 256, 512} x H = W in {20, 40, 80, 160} x batch in {1, 32} x k in {2, 3, 4, 9} x {bf16, fp32}.

For every point: cold-L2 and warm kernel time (CUDA events), algorithmic GB/s, non-zero GFLOP/s and the
fraction of the point's roofline max(bytes / HBM peak, nnz FLOP / pipe peak).  Both types run NHWC on the tensor
path where it applies (fp32: kind::tf32 with three products per tap, pipe peak = bf16 peak / 2 / 3); `--fp32-nchw`
runs fp32 in NCHW on the FMA pipes instead.  Writes a CSV and prints a short summary.

    python -m paper_2303_02191_b200.sweep --out sweep.csv [--quick]
"""
import argparse
import csv
import json
import os

import numpy as np

from . import synth

ALU_PEAK_TFLOPS = 148 * 128 * 2 * 1.965e9 / 1e12   # FP32 FMA pipes at the maximum SM clock


def peaks():
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    try:
        d = json.load(open(os.path.join(root, "MEASURED_PEAKS.json")))
        return float(d["hbm_gbs"]), float(d["bf16_tflops"]), "measured"
    except Exception:
        return 6650.0, 1590.0, "fallback"


def points(quick):
    cs, hs, ns, ks = (64, 256, 512), (20, 40, 80, 160), (1, 32), (2, 3, 4, 9)
    if quick:
        cs, hs, ns, ks = (64, 256), (20, 80), (1,), (3, 9)
    for dt in ("bf16", "f32"):
        for c in cs:
            for h in hs:
                for n in ns:
                    for k in ks:
                        yield dt, c, h, n, k


def main():
    import torch
    from . import binding as rt

    ap = argparse.ArgumentParser()
    ap.add_argument("--out", default="sweep.csv")
    ap.add_argument("--quick", action="store_true")
    ap.add_argument("--reps", type=int, default=10)
    ap.add_argument("--fp32-nchw", action="store_true", help="fp32 points in NCHW on the FMA path")
    ap.add_argument("--only", default=None, help="bf16 or f32: only that half of the sweep")
    args = ap.parse_args()
    hbm, tc_peak, kind = peaks()
    ctx = rt.Context(0)
    dev = torch.device("cuda", 0)
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)
    rows = []
    for dt, C, H, N, k in points(args.quick):
        if args.only and dt != args.only:
            continue
        tdt = torch.bfloat16 if dt == "bf16" else torch.float32
        layout = rt.NCHW if (dt == "f32" and args.fp32_nchw) else rt.NHWC
        preset = {2: rt.PRESET_CONN4, 3: rt.PRESET_CONN4, 4: rt.PRESET_CENTRE8, 9: rt.PRESET_DENSE}[k]
        masks = rt.rtoss_pattern_preset(k, preset)
        w = torch.from_numpy(synth.kaiming_weights(0, C + k, C, C, 3)).to(dev)
        b = torch.from_numpy(synth.bias(0, C, C)).to(dev)
        pid = ctx.rtoss_select_patterns(w, 3, masks, k)
        packed = ctx.rtoss_pack(w, 3, masks, k, pid, rt.DTYPE_NAMES[dt])
        shape = (N, H, H, C) if layout == rt.NHWC else (N, C, H, H)
        x = torch.randn(shape, device=dev, dtype=torch.float32).to(tdt)
        y = torch.empty(shape, device=dev, dtype=tdt)
        path = rt.PATH_TENSOR
        try:
            ctx.rtoss_conv3x3_pattern(packed, x, y, N, H, H, 1, layout, rt.ACT_SILU, b, path=path)
        except rt.RtossError as err:
            if err.status != 3:
                raise
            path = rt.PATH_FMA
        torch.cuda.synchronize()
        reps = args.reps if N * C * C * H * H < 2e11 else 3
        ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(2 * reps)]
        for i in range(reps):                       # cold: a 256 MB write before every launch
            flush.zero_()
            ev[i][0].record()
            ctx.rtoss_conv3x3_pattern(packed, x, y, N, H, H, 1, layout, rt.ACT_SILU, b, path=path)
            ev[i][1].record()
        ev[reps][0].record()
        for i in range(reps):                       # warm: back to back
            ctx.rtoss_conv3x3_pattern(packed, x, y, N, H, H, 1, layout, rt.ACT_SILU, b, path=path)
        ev[reps][1].record()
        torch.cuda.synchronize()
        cold = float(np.median([a.elapsed_time(b_) for a, b_ in ev[:reps]]))
        warm = ev[reps][0].elapsed_time(ev[reps][1]) / reps
        L = dict(ksize=3, stride=1, cin=C, cout=C, H=H, W=H)
        flops = synth.layer_nnz_flops(L, N, k)
        nbytes = synth.layer_bytes(L, N, k, 2 if dt == "bf16" else 4)
        # tensor pipe: measured bf16 peak; fp32 runs tf32 instructions (half the rate) three times per product
        pipe = (tc_peak if dt == "bf16" else tc_peak / 6) if path == rt.PATH_TENSOR else ALU_PEAK_TFLOPS
        t_roof = max(nbytes / (hbm * 1e9), flops / (pipe * 1e12))
        rows.append(dict(dtype=dt, C=C, HW=H, N=N, k=k, path="tensor" if path == rt.PATH_TENSOR else "fma",
                         cold_ms=round(cold, 5), warm_ms=round(warm, 5), gbs=round(nbytes / cold / 1e6, 1),
                         nnz_gflops=round(flops / cold / 1e6, 1), roofline_us=round(t_roof * 1e6, 2),
                         bound="hbm" if nbytes / (hbm * 1e9) >= flops / (pipe * 1e12) else
                         (("tensor" if dt == "bf16" else "tensor (tf32 x3)") if path == rt.PATH_TENSOR else "alu"),
                         frac=round(t_roof / (cold * 1e-3), 4)))
        packed.close()
        del x, y
    assert ctx.rtoss_device_status() == 0
    os.makedirs(os.path.dirname(os.path.abspath(args.out)), exist_ok=True)
    with open(args.out, "w", newline="") as f:
        wr = csv.DictWriter(f, fieldnames=list(rows[0].keys()))
        wr.writeheader()
        wr.writerows(rows)
    for dt in ("bf16", "f32"):
        sel = [r for r in rows if r["dtype"] == dt]
        if not sel:
            continue
        fr = np.array([r["frac"] for r in sel])
        best = max(sel, key=lambda r: r["frac"])
        print("%s: %d points, roofline fraction median %.3f, max %.3f (C=%d HW=%d N=%d k=%d, %.1f nnz GFLOP/s); peaks %s" %
              (dt, len(sel), float(np.median(fr)), float(fr.max()), best["C"], best["HW"], best["N"], best["k"],
               best["nnz_gflops"], kind))
    ctx.close()


if __name__ == "__main__":
    main()
