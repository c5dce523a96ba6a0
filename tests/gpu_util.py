"""Helpers of the GPU parity tests: run one layer through the C-ABI library and
through the CPU oracle on the same seeded inputs."""
import numpy as np
import torch

from oracle import rtoss_oracle as orc
from paper_2303_02191_b200 import binding as rt
from paper_2303_02191_b200 import synth

TORCH_DT = {"f32": torch.float32, "bf16": torch.bfloat16, "f16": torch.float16}
ORC_DT = {"f32": orc.DT_F32, "bf16": orc.DT_BF16, "f16": orc.DT_F16}
TOL = {"f32": 1e-4, "bf16": 2e-2, "f16": 2e-2}   # max relative error allowed (fp32 accumulate on the GPU)

_ctx = None


def ctx():
    global _ctx
    if _ctx is None:
        _ctx = rt.Context(0)
    return _ctx


def to_dev(a, dt, layout="nchw"):
    t = torch.from_numpy(np.ascontiguousarray(a)).to(TORCH_DT[dt])
    if layout == "nhwc" and t.dim() == 4:
        t = t.permute(0, 2, 3, 1).contiguous()
    return t.cuda()


def from_dev(t, layout="nchw"):
    t = t.float().cpu()
    if layout == "nhwc" and t.dim() == 4:
        t = t.permute(0, 3, 1, 2).contiguous()
    return t.numpy()


def select_pack(w, ksize, masks, k, dt, w_dt="f32"):
    """-> (pid numpy, packed handle, export dict).  w numpy fp32 [Cout,Cin,ks,ks]."""
    c = ctx()
    wd = to_dev(synth.round_like(w, w_dt), w_dt)
    pid = c.rtoss_select_patterns(wd, ksize, masks, k)
    packed = c.rtoss_pack(wd, ksize, masks, k, pid, rt.DTYPE_NAMES[dt])
    torch.cuda.synchronize()
    return pid.cpu().numpy(), packed


def oracle_weights(w, ksize, masks, k, dt, w_dt="f32"):
    """Oracle side of select+pack -> (pid, dense masked weights rounded to dt, pack arrays)."""
    wr = synth.round_like(w, w_dt)
    if ksize == 3:
        pid = orc.select_3x3(wr, masks)
        val, perm, off = orc.pack_3x3(wr, masks, k, pid, ORC_DT[dt])
        wd = orc.unpack_3x3(val, w.shape[0], w.shape[1], masks, k, pid)
        return pid, wd, dict(val=val, perm=perm, bucket_off=off)
    w2 = wr.reshape(w.shape[0], w.shape[1])
    pid = orc.select_1x1(w2, masks)
    val = orc.pack_1x1(w2, masks, k, pid, ORC_DT[dt])
    wd = orc.unpack_1x1(val, w.shape[0], w.shape[1], masks, k, pid)
    return pid, wd, dict(val=val)


def val_as_f32(exported_val, dt):
    if dt == "f32":
        return exported_val
    t = torch.from_numpy(exported_val.view(np.int16).copy()).view(TORCH_DT[dt])
    return t.float().numpy()


def run_conv(packed, ksize, x, dt, stride, act, bias, layout="nchw", y_off=0, y_stride=0, host=False, path=0):
    """x numpy fp32 NCHW (already rounded to dt) -> y numpy fp32 NCHW."""
    c = ctx()
    N, Cin, H, W = x.shape
    Cout = packed.info.Cout
    Ho, Wo = synth.out_hw(H, W, stride)
    Cs = y_stride if y_stride else Cout
    lay = rt.NHWC if layout == "nhwc" else rt.NCHW
    bd = torch.from_numpy(bias).cuda() if bias is not None else None
    yshape = (N, Ho, Wo, Cs) if layout == "nhwc" else (N, Cs, Ho, Wo)
    if host:
        xh = to_dev(x, dt, layout).cpu().pin_memory()
        yh = torch.full(yshape, 7.0, dtype=TORCH_DT[dt]).pin_memory()
        torch.cuda.synchronize()
        c.rtoss_conv_pattern_host(packed, xh, yh, N, H, W, stride, lay, rt.ACT_NAMES[act], bd, y_off, y_stride, path)
        return from_dev(yh, layout)
    xd = to_dev(x, dt, layout)
    yd = torch.full(yshape, 7.0, dtype=TORCH_DT[dt], device="cuda")
    fn = c.rtoss_conv3x3_pattern if ksize == 3 else c.rtoss_conv1x1_pattern
    fn(packed, xd, yd, N, H, W, stride, lay, rt.ACT_NAMES[act], bd, y_off, y_stride, path)
    torch.cuda.synchronize()
    return from_dev(yd, layout)


def oracle_conv(ksize, x, wd, bias, stride, act, dt):
    a = {"none": orc.ACT_NONE, "relu": orc.ACT_RELU, "silu": orc.ACT_SILU}[act]
    fn = orc.conv3x3 if ksize == 3 else orc.conv1x1
    return fn(x, wd, bias, stride, a, ORC_DT[dt])


def check_layer(seed, tid, ksize, N, Cin, Cout, H, W, stride, k, masks, dt, act="none", layout="nchw",
                use_bias=True, host=False, path=0):
    """Full parity of one layer: pattern ids and packed arrays bit-exact, outputs within TOL[dt]."""
    x = synth.round_like(synth.activations(seed, tid, N, Cin, H, W), dt)
    w = synth.kaiming_weights(seed, tid, Cout, Cin, ksize)
    b = synth.bias(seed, tid, Cout) if use_bias else None
    pid_g, packed = select_pack(w, ksize, masks, k, dt)
    pid_o, wd, arrays = oracle_weights(w, ksize, masks, k, dt)
    assert np.array_equal(pid_g, pid_o.ravel()), "pattern ids differ"
    ex = packed.export()
    assert np.array_equal(ex["pid"], pid_o.ravel())
    assert np.array_equal(val_as_f32(ex["val"], dt).view(np.uint32), arrays["val"].view(np.uint32)), "packed values differ"
    if ksize == 3:
        assert np.array_equal(ex["perm"], arrays["perm"]) and np.array_equal(ex["bucket_off"], arrays["bucket_off"])
    y = run_conv(packed, ksize, x, dt, stride, act, b, layout, host=host, path=path)
    ref = oracle_conv(ksize, x, wd, b, stride, act, dt)
    err = orc.rel_err(y, ref)
    assert y.shape == ref.shape
    assert err <= TOL[dt], "relative error %.3g above %.3g" % (err, TOL[dt])
    packed.close()
    return err
