"""ctypes front end of the R-TOSS CPU oracle (``rtoss_oracle.c``).

TEST INFRASTRUCTURE, NOT A PRODUCT PATH: only the tests, the smoke check and
the benchmark's CPU-baseline / reference legs may import this module.  It
shares nothing with the CUDA library.  Arrays are numpy, float32 unless
stated; activations are NCHW.  ``build()`` compiles the C file with gcc.
"""
import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "rtoss_oracle.c")
_LIB = os.path.join(_HERE, "librtoss_oracle.so")

PRESET_ALL, PRESET_CONN4, PRESET_CENTRE8, PRESET_DENSE = 0, 1, 2, 3
DT_F32, DT_BF16, DT_F16 = 0, 1, 2
ACT_NONE, ACT_RELU, ACT_SILU = 0, 1, 2

_lib = None


def build(force=False):
    """Compile the oracle (gcc, OpenMP, no FP contraction)."""
    import hashlib
    stamp = _LIB + ".stamp"
    fp = hashlib.sha256(open(_SRC, "rb").read()).hexdigest()
    if force or not os.path.exists(_LIB) or not os.path.exists(stamp) or open(stamp).read().strip() != fp:
        cmd = ["gcc", "-O2", "-std=c11", "-fopenmp", "-ffp-contract=off", "-fPIC", "-shared",
               _SRC, "-o", _LIB, "-lm"]
        subprocess.check_call(cmd)
        open(stamp, "w").write(fp)
    return _LIB


def lib():
    global _lib
    if _lib is None:
        build()
        _lib = ctypes.CDLL(_LIB)
        _lib.oracle_select_1x1.restype = ctypes.c_long
        _lib.oracle_round_to.restype = ctypes.c_float
        _lib.oracle_round_to.argtypes = [ctypes.c_float, ctypes.c_int]
        _lib.oracle_f32_to_bf16_bits.restype = ctypes.c_uint16
        _lib.oracle_f32_to_bf16_bits.argtypes = [ctypes.c_float]
        _lib.oracle_f32_to_f16_bits.restype = ctypes.c_uint16
        _lib.oracle_f32_to_f16_bits.argtypes = [ctypes.c_float]
    return _lib


def _p(a):
    return a.ctypes.data_as(ctypes.c_void_p) if a is not None else None


def _f32(a):
    return np.ascontiguousarray(a, dtype=np.float32)


def _masks(m):
    return np.ascontiguousarray(m, dtype=np.uint16)


def pattern_preset(k, preset):
    out = np.zeros(512, dtype=np.uint16)
    n = lib().oracle_pattern_preset(int(k), int(preset), _p(out), 512)
    if n < 0:
        raise ValueError("bad preset arguments")
    return out[:n].copy()


def pattern_table_valid(masks, k):
    m = _masks(masks)
    return bool(lib().oracle_pattern_table_valid(_p(m), len(m), int(k)))


def select_kernels(w9, masks):
    """w9: [..., 9] -> uint8 pattern id per kernel (Algorithm 2)."""
    w9 = _f32(w9).reshape(-1, 9)
    m = _masks(masks)
    pid = np.zeros(w9.shape[0], dtype=np.uint8)
    lib().oracle_select_kernels(_p(w9), ctypes.c_long(w9.shape[0]), _p(m), len(m), _p(pid))
    return pid


def pattern_usage(w9, masks):
    """Section IV.B, criterion 2: how many kernels of the sample choose each candidate pattern (Algorithm 2's argmax
    per kernel, then a plain count)."""
    m = _masks(masks)
    counts = np.zeros(len(m), dtype=np.uint64)
    for p in select_kernels(w9, m):
        counts[p] += 1
    return counts


def pattern_rank(masks, counts, M):
    """The cut of criterion 2: candidates by falling count, equal counts by rising mask value; the M best, returned in
    ascending mask order (a table).  Also returns the candidate indices in rank order."""
    m = [int(v) for v in _masks(masks)]
    c = [int(v) for v in counts]
    order = sorted(range(len(m)), key=lambda i: (-c[i], m[i]))
    top = sorted(m[i] for i in order[:M])
    return np.array(top, dtype=np.uint16), np.array(order, dtype=np.int32)


def derive_pattern_table(w9, k, preset, M):
    """Section IV.B end to end: Eq. 1 candidates (preset ALL) or those with adjacent taps (preset CONN4), usage over
    the sample, the M most used."""
    cand = pattern_preset(k, preset)
    counts = pattern_usage(w9, cand)
    top, _ = pattern_rank(cand, counts, min(M, len(cand)))
    return top, cand, counts


def select_3x3(w, masks):
    w = _f32(w)
    Cout, Cin = w.shape[:2]
    m = _masks(masks)
    pid = np.zeros((Cout, Cin), dtype=np.uint8)
    lib().oracle_select_3x3(_p(w), Cout, Cin, _p(m), len(m), _p(pid))
    return pid


def select_shared(w, masks, FB, CB):
    """One pattern per block of FB filters x CB input channels: the pattern retaining the most energy of the block
    (a variant of Algorithm 2, see the C source).  w [Cout, Cin, 3, 3] -> pid [Cout, Cin], constant per block."""
    w = _f32(w)
    Cout, Cin = w.shape[:2]
    m = _masks(masks)
    pid = np.zeros((Cout, Cin), dtype=np.uint8)
    lib().oracle_select_shared(_p(w), Cout, Cin, int(FB), int(CB), _p(m), len(m), _p(pid))
    return pid


def select_1x1(w, masks):
    """w: [Cout, Cin] -> pid1[G], G = floor(Cout*Cin/9) (Algorithm 3)."""
    w = _f32(w).reshape(w.shape[0], -1)
    Cout, Cin = w.shape
    m = _masks(masks)
    pid1 = np.zeros(max((Cout * Cin) // 9, 1), dtype=np.uint8)
    G = lib().oracle_select_1x1(_p(w), Cout, Cin, _p(m), len(m), _p(pid1))
    return pid1[:G].copy()


def mask_3x3(w, masks, pid):
    w = _f32(w)
    Cout, Cin = w.shape[:2]
    m = _masks(masks)
    pid = np.ascontiguousarray(pid, dtype=np.uint8)
    out = np.empty_like(w)
    lib().oracle_mask_3x3(_p(w), Cout, Cin, _p(m), _p(pid), _p(out))
    return out


def mask_1x1(w, masks, pid1):
    w = _f32(w).reshape(w.shape[0], -1)
    Cout, Cin = w.shape
    m = _masks(masks)
    pid1 = np.ascontiguousarray(pid1, dtype=np.uint8)
    out = np.empty_like(w)
    lib().oracle_mask_1x1(_p(w), Cout, Cin, _p(m), _p(pid1), _p(out))
    return out


def round_array(a, dtype):
    a = _f32(a)
    out = np.empty_like(a)
    lib().oracle_round_array(_p(a), ctypes.c_long(a.size), int(dtype), _p(out))
    return out


def f32_to_bf16_bits(v):
    return int(lib().oracle_f32_to_bf16_bits(float(v)))


def f32_to_f16_bits(v):
    return int(lib().oracle_f32_to_f16_bits(float(v)))


def pack_3x3(w, masks, k, pid, compute_dtype):
    """-> (val[Cout*Cin*k] float32 holding the rounded values, perm, bucket_off)."""
    w = _f32(w)
    Cout, Cin = w.shape[:2]
    m = _masks(masks)
    P = len(m)
    pid = np.ascontiguousarray(pid, dtype=np.uint8)
    val = np.zeros(Cout * Cin * k, dtype=np.float32)
    perm = np.zeros(Cin * Cout, dtype=np.uint32)
    off = np.zeros(Cin * (P + 1), dtype=np.uint32)
    lib().oracle_pack_3x3(_p(w), Cout, Cin, _p(m), P, int(k), _p(pid), int(compute_dtype), _p(val), _p(perm), _p(off))
    return val, perm, off


def pack_1x1(w, masks, k, pid1, compute_dtype):
    w = _f32(w).reshape(w.shape[0], -1)
    Cout, Cin = w.shape
    m = _masks(masks)
    pid1 = np.ascontiguousarray(pid1, dtype=np.uint8)
    G = (Cout * Cin) // 9
    val1 = np.zeros(max(G * k, 1), dtype=np.float32)
    lib().oracle_pack_1x1(_p(w), Cout, Cin, _p(m), int(k), _p(pid1), int(compute_dtype), _p(val1))
    return val1[:G * k].copy()


def unpack_3x3(val, Cout, Cin, masks, k, pid):
    m = _masks(masks)
    val = _f32(val)
    pid = np.ascontiguousarray(pid, dtype=np.uint8)
    wd = np.empty((Cout, Cin, 3, 3), dtype=np.float32)
    lib().oracle_unpack_3x3(_p(val), Cout, Cin, _p(m), int(k), _p(pid), _p(wd))
    return wd


def unpack_1x1(val1, Cout, Cin, masks, k, pid1):
    m = _masks(masks)
    val1 = _f32(val1)
    pid1 = np.ascontiguousarray(pid1, dtype=np.uint8)
    wd = np.empty((Cout, Cin), dtype=np.float32)
    lib().oracle_unpack_1x1(_p(val1), Cout, Cin, _p(m), int(k), _p(pid1), _p(wd))
    return wd


def _out_hw(H, W, stride):
    return (H - 1) // stride + 1, (W - 1) // stride + 1


def conv3x3(x, wd, bias, stride, act, out_dtype):
    """x [N,Cin,H,W]; wd [Cout,Cin,3,3] already masked and rounded -> y [N,Cout,Ho,Wo]."""
    x, wd = _f32(x), _f32(wd)
    N, Cin, H, W = x.shape
    Cout = wd.shape[0]
    Ho, Wo = _out_hw(H, W, stride)
    b = _f32(bias) if bias is not None else None
    y = np.empty((N, Cout, Ho, Wo), dtype=np.float32)
    lib().oracle_conv3x3(_p(x), N, Cin, H, W, _p(wd), Cout, _p(b), int(stride), int(act), int(out_dtype), _p(y))
    return y


def conv1x1(x, wd, bias, stride, act, out_dtype):
    x, wd = _f32(x), _f32(wd).reshape(wd.shape[0], -1)
    N, Cin, H, W = x.shape
    Cout = wd.shape[0]
    Ho, Wo = _out_hw(H, W, stride)
    b = _f32(bias) if bias is not None else None
    y = np.empty((N, Cout, Ho, Wo), dtype=np.float32)
    lib().oracle_conv1x1(_p(x), N, Cin, H, W, _p(wd), Cout, _p(b), int(stride), int(act), int(out_dtype), _p(y))
    return y


def conv_points(ksize, x, wd, bias, stride, act, out_dtype, idx):
    """Selected outputs only; idx int32 [npts,4] rows (n, co, oy, ox)."""
    x, wd = _f32(x), _f32(wd)
    N, Cin, H, W = x.shape
    Cout = wd.shape[0]
    b = _f32(bias) if bias is not None else None
    idx = np.ascontiguousarray(idx, dtype=np.int32)
    out = np.empty(idx.shape[0], dtype=np.float32)
    fn = lib().oracle_conv3x3_points if ksize == 3 else lib().oracle_conv1x1_points
    fn(_p(x), N, Cin, H, W, _p(wd), Cout, _p(b), int(stride), int(act), int(out_dtype), _p(idx),
       ctypes.c_long(idx.shape[0]), _p(out))
    return out


def group_layers(nodes):
    """nodes: list of dicts {kind: 'conv'|'op', cout, cin, ksize, inputs: [ids]} in
    topological order -> (parent, group, ngroups) (Algorithm 1)."""
    L = len(nodes)
    kind = np.array([1 if n["kind"] == "conv" else 0 for n in nodes], dtype=np.int32)
    cout = np.array([n.get("cout", 0) for n in nodes], dtype=np.int32)
    cin = np.array([n.get("cin", 0) for n in nodes], dtype=np.int32)
    ks = np.array([n.get("ksize", 0) for n in nodes], dtype=np.int32)
    in_off = np.zeros(L + 1, dtype=np.int32)
    flat = []
    for i, n in enumerate(nodes):
        flat.extend(n.get("inputs", []))
        in_off[i + 1] = len(flat)
    in_idx = np.array(flat if flat else [0], dtype=np.int32)
    parent = np.zeros(L, dtype=np.int32)
    group = np.zeros(L, dtype=np.int32)
    ng = lib().oracle_group_layers(L, _p(kind), _p(cout), _p(cin), _p(ks), _p(in_off), _p(in_idx), _p(parent), _p(group))
    return parent, group, ng


def rel_err(y, y_ref):
    """max |y - y_ref| / max(|y_ref|, rms(y_ref)) over the tensor."""
    y = np.asarray(y, dtype=np.float64)
    r = np.asarray(y_ref, dtype=np.float64)
    rms = float(np.sqrt(np.mean(r * r))) if r.size else 0.0
    den = np.maximum(np.abs(r), max(rms, 1e-30))
    return float(np.max(np.abs(y - r) / den)) if r.size else 0.0


def maxpool2d(x, k, stride, pad):
    x = _f32(x)
    N, C, H, W = x.shape
    Ho, Wo = (H + 2 * pad - k) // stride + 1, (W + 2 * pad - k) // stride + 1
    y = np.empty((N, C, Ho, Wo), dtype=np.float32)
    lib().oracle_maxpool2d(_p(x), N, C, H, W, int(k), int(stride), int(pad), _p(y))
    return y


def upsample2x(x):
    x = _f32(x)
    N, C, H, W = x.shape
    y = np.empty((N, C, 2 * H, 2 * W), dtype=np.float32)
    lib().oracle_upsample2x(_p(x), N, C, H, W, _p(y))
    return y


def add_act(a, b, act, out_dtype):
    a, b = _f32(a), _f32(b)
    y = np.empty_like(a)
    lib().oracle_add_act(_p(a), _p(b), ctypes.c_long(a.size), int(act), int(out_dtype), _p(y))
    return y
