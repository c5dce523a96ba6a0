"""ctypes binding of ``librtoss.so`` (declared in ``include/rtoss.h``).

Argument marshalling only: every step runs in the library's CUDA kernels.
Importing this module loads the library and raises ``RuntimeError`` when it is
missing; there is no CPU fallback.  Tensors are torch CUDA tensors (torch is
used for device memory and streams only).
"""
import ctypes
import os

import numpy as np

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG, "librtoss.so")

OK = 0
ERR_UNSUPPORTED = 3
F32, BF16, F16 = 0, 1, 2
NCHW, NHWC = 0, 1
ACT_NONE, ACT_RELU, ACT_SILU = 0, 1, 2
PRESET_ALL, PRESET_CONN4, PRESET_CENTRE8, PRESET_DENSE = 0, 1, 2, 3
PATH_AUTO, PATH_FMA, PATH_TENSOR = 0, 1, 2
DTYPE_NAMES = {"f32": F32, "bf16": BF16, "f16": F16}
ACT_NAMES = {"none": ACT_NONE, "relu": ACT_RELU, "silu": ACT_SILU}

SYMBOLS = [
    "rtoss_create", "rtoss_destroy", "rtoss_status_string", "rtoss_last_error", "rtoss_pattern_preset",
    "rtoss_pattern_table_validate", "rtoss_group_layers", "rtoss_select_patterns", "rtoss_pack",
    "rtoss_packed_info_get", "rtoss_packed_export", "rtoss_packed_to_dense", "rtoss_packed_destroy",
    "rtoss_conv3x3_pattern", "rtoss_conv1x1_pattern", "rtoss_conv_pattern_host", "rtoss_device_status", "rtoss_prune_dense_static", "rtoss_maxpool2d", "rtoss_upsample2x", "rtoss_add_act", "rtoss_pattern_usage",
    "rtoss_pattern_rank", "rtoss_pattern_table_derive",
    "rtoss_batch_create", "rtoss_batch_select_pack", "rtoss_batch_destroy",
    "rtoss_select_patterns_shared", "rtoss_conv_group", "rtoss_set_wait_limit", "rtoss_inject_lost_copy",
    "rtoss_fma_plan3x3", "rtoss_conv_chain", "rtoss_chain_deps", "rtoss_chain_deps_spans", "rtoss_tensor_plan_of",
]


class RtossError(RuntimeError):
    def __init__(self, status, text):
        super().__init__("rtoss status %d: %s" % (status, text))
        self.status = status


class LayerNode(ctypes.Structure):
    _fields_ = [("is_conv", ctypes.c_int), ("cout", ctypes.c_int), ("cin", ctypes.c_int), ("ksize", ctypes.c_int),
                ("n_inputs", ctypes.c_int), ("inputs", ctypes.POINTER(ctypes.c_int))]


class PackedInfo(ctypes.Structure):
    _fields_ = [("Cout", ctypes.c_int), ("Cin", ctypes.c_int), ("ksize", ctypes.c_int), ("P", ctypes.c_int),
                ("k", ctypes.c_int), ("dtype", ctypes.c_int), ("n_kernels", ctypes.c_int64),
                ("n_values", ctypes.c_int64)]


class BatchItem(ctypes.Structure):
    _fields_ = [("w_dev", ctypes.c_void_p), ("w_dtype", ctypes.c_int), ("Cout", ctypes.c_int), ("Cin", ctypes.c_int),
                ("ksize", ctypes.c_int), ("masks_host", ctypes.c_void_p), ("P", ctypes.c_int), ("k", ctypes.c_int),
                ("pid_dev", ctypes.c_void_p), ("packed", ctypes.c_void_p), ("pid_from", ctypes.c_int)]


class ConvDesc(ctypes.Structure):
    _fields_ = [("N", ctypes.c_int), ("H", ctypes.c_int), ("W", ctypes.c_int), ("stride", ctypes.c_int),
                ("layout", ctypes.c_int), ("io_dtype", ctypes.c_int), ("act", ctypes.c_int),
                ("bias_dev", ctypes.c_void_p), ("y_channel_offset", ctypes.c_int), ("y_channel_stride", ctypes.c_int),
                ("path", ctypes.c_int), ("residual_dev", ctypes.c_void_p), ("residual_after_act", ctypes.c_int)]


class FmaPlan(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int) for n in (
        "small_cin", "pixels_per_lane", "filters_per_warp", "warps", "ctas_per_sm", "lanes_x", "lanes_y", "tiles_x", "tiles_y",
        "grid_x", "grid_y", "staged_rows", "staged_cols", "staging", "vector_bytes", "vectors_per_plane", "shared_bytes")]


class TensorPlan(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int) for n in (
        "eligible", "rows_per_tile", "cols_per_tile", "pitch", "positions", "staged_rows", "sub_tiles", "act_stages",
        "weight_stages", "taps_per_weight_stage", "row_bytes", "act_stage_bytes", "weight_stage_bytes", "shared_bytes",
        "positions_on_m", "split_k", "tiles")]


class ConvItem(ctypes.Structure):
    _fields_ = [("packed", ctypes.c_void_p), ("x_dev", ctypes.c_void_p), ("y_dev", ctypes.c_void_p), ("desc", ConvDesc)]


def _load():
    if not os.path.exists(LIB_PATH):
        raise RuntimeError("librtoss.so not built (%s): run `python -m paper_2303_02191_b200._build`; "
                           "there is no CPU fallback" % LIB_PATH)
    lib = ctypes.CDLL(LIB_PATH)
    vp, ci = ctypes.c_void_p, ctypes.c_int
    lib.rtoss_create.argtypes = [ci, ctypes.POINTER(vp)]
    lib.rtoss_destroy.argtypes = [vp]
    lib.rtoss_destroy.restype = None
    lib.rtoss_status_string.argtypes = [ci]
    lib.rtoss_status_string.restype = ctypes.c_char_p
    lib.rtoss_last_error.argtypes = [vp]
    lib.rtoss_last_error.restype = ctypes.c_char_p
    lib.rtoss_pattern_preset.argtypes = [ci, ci, vp, ctypes.POINTER(ci)]
    lib.rtoss_pattern_table_validate.argtypes = [vp, ci, ci]
    lib.rtoss_pattern_rank.argtypes = [vp, vp, ci, ci, ci, vp, vp]
    lib.rtoss_pattern_table_derive.argtypes = [vp, vp, ci, ctypes.c_int64, ci, ci, ci, vp, vp, vp, ctypes.POINTER(ci), vp, vp,
                                               ctypes.POINTER(ci), vp]
    lib.rtoss_group_layers.argtypes = [ctypes.POINTER(LayerNode), ci, vp, vp, ctypes.POINTER(ci)]
    lib.rtoss_select_patterns.argtypes = [vp, vp, ci, ci, ci, ci, vp, ci, ci, vp, vp]
    lib.rtoss_pack.argtypes = [vp, vp, ci, ci, ci, ci, vp, ci, ci, vp, ci, ctypes.POINTER(vp), vp]
    lib.rtoss_packed_info_get.argtypes = [vp, ctypes.POINTER(PackedInfo)]
    lib.rtoss_packed_export.argtypes = [vp, vp, vp, vp, vp, vp, vp]
    lib.rtoss_packed_to_dense.argtypes = [vp, vp, vp, vp]
    lib.rtoss_packed_destroy.argtypes = [vp]
    lib.rtoss_packed_destroy.restype = None
    lib.rtoss_conv3x3_pattern.argtypes = [vp, vp, vp, vp, ctypes.POINTER(ConvDesc), vp]
    lib.rtoss_conv1x1_pattern.argtypes = [vp, vp, vp, vp, ctypes.POINTER(ConvDesc), vp]
    lib.rtoss_conv_pattern_host.argtypes = [vp, vp, vp, vp, ctypes.POINTER(ConvDesc)]
    lib.rtoss_device_status.argtypes = [vp, ctypes.POINTER(ci)]
    lib.rtoss_conv_group.argtypes = [vp, ctypes.POINTER(ConvItem), ci, ctypes.POINTER(ci), vp]
    lib.rtoss_conv_chain.argtypes = [vp, ctypes.POINTER(ConvItem), ci, ctypes.POINTER(ctypes.c_uint32), ctypes.POINTER(ci), vp]
    lib.rtoss_chain_deps.argtypes = [ctypes.POINTER(ConvItem), ci, ctypes.POINTER(ctypes.c_uint32)]
    lib.rtoss_tensor_plan_of.argtypes = [ctypes.POINTER(ConvDesc), ci, ci, ci, ci, ci, ctypes.POINTER(TensorPlan)]
    lib.rtoss_chain_deps_spans.argtypes = [ctypes.POINTER(ctypes.c_uint64), ci, ctypes.POINTER(ctypes.c_uint32)]
    lib.rtoss_set_wait_limit.argtypes = [vp, ctypes.c_longlong]
    lib.rtoss_inject_lost_copy.argtypes = [vp]
    lib.rtoss_fma_plan3x3.argtypes = [ctypes.POINTER(ConvDesc), ci, ci, ci, ci, ctypes.POINTER(FmaPlan)]
    lib.rtoss_select_patterns_shared.argtypes = [vp, vp, ci, ci, ci, ci, ci, vp, ci, ci, vp, vp]
    lib.rtoss_prune_dense_static.argtypes = [vp, ci, ci, ci, ci, vp, ci, ci, vp, vp]
    lib.rtoss_maxpool2d.argtypes = [vp, vp, ci, ci, ci, ci, ci, ci, ci, ci, ci, ci, ci, vp]
    lib.rtoss_upsample2x.argtypes = [vp, vp, ci, ci, ci, ci, ci, ci, ci, ci, vp]
    lib.rtoss_add_act.argtypes = [vp, vp, vp, ctypes.c_int64, ci, ci, vp]
    lib.rtoss_pattern_usage.argtypes = [vp, vp, ci, ctypes.c_int64, vp, ci, ci, vp, vp, vp]
    lib.rtoss_batch_create.argtypes = [vp, ctypes.POINTER(BatchItem), ci, ctypes.POINTER(vp)]
    lib.rtoss_batch_select_pack.argtypes = [vp, vp, vp]
    lib.rtoss_batch_destroy.argtypes = [vp]
    lib.rtoss_batch_destroy.restype = None
    return lib


lib = _load()


def status_string(s):
    return lib.rtoss_status_string(int(s)).decode()


def _masks_arr(masks):
    return np.ascontiguousarray(masks, dtype=np.uint16)


def _np_ptr(a):
    return a.ctypes.data_as(ctypes.c_void_p)


def rtoss_pattern_preset(k, preset):
    """-> numpy uint16 masks (host only)."""
    out = np.zeros(512, dtype=np.uint16)
    n = ctypes.c_int(512)
    st = lib.rtoss_pattern_preset(int(k), int(preset), _np_ptr(out), ctypes.byref(n))
    if st != OK:
        raise RtossError(st, status_string(st))
    return out[:n.value].copy()


def rtoss_pattern_rank(masks, counts, k, M):
    """-> (the M most used masks in ascending order, candidate indices in rank order); host only."""
    m = _masks_arr(masks)
    c = np.ascontiguousarray(counts, dtype=np.uint64)
    top = np.zeros(max(int(M), 1), dtype=np.uint16)
    order = np.zeros(len(m), dtype=np.int32)
    st = lib.rtoss_pattern_rank(_np_ptr(m), _np_ptr(c), len(m), int(k), int(M), _np_ptr(top), _np_ptr(order))
    if st != OK:
        raise RtossError(st, status_string(st))
    return top[:int(M)].copy(), order


def rtoss_pattern_table_validate(masks, k):
    m = _masks_arr(masks)
    return lib.rtoss_pattern_table_validate(_np_ptr(m), len(m), int(k))


def rtoss_group_layers(nodes):
    """nodes: list of dict(kind, cout, cin, ksize, inputs) -> (parent, group, n_groups) (host only)."""
    L = len(nodes)
    arr = (LayerNode * max(L, 1))()
    keep = []
    for i, nd in enumerate(nodes):
        ins = list(nd.get("inputs", []))
        buf = (ctypes.c_int * max(len(ins), 1))(*ins)
        keep.append(buf)
        arr[i] = LayerNode(1 if nd["kind"] == "conv" else 0, nd.get("cout", 0), nd.get("cin", 0), nd.get("ksize", 0),
                           len(ins), ctypes.cast(buf, ctypes.POINTER(ctypes.c_int)))
    parent = np.zeros(max(L, 1), dtype=np.int32)
    group = np.zeros(max(L, 1), dtype=np.int32)
    ng = ctypes.c_int(0)
    st = lib.rtoss_group_layers(arr, L, _np_ptr(parent), _np_ptr(group), ctypes.byref(ng))
    if st != OK:
        raise RtossError(st, status_string(st))
    return parent[:L], group[:L], ng.value


def _glue_check(st):
    if st != OK:
        raise RtossError(st, status_string(st))


def rtoss_maxpool2d(x, y, N, C, H, W, k, stride, pad, layout=NCHW, y_channel_offset=0, y_channel_stride=0):
    _glue_check(lib.rtoss_maxpool2d(x.data_ptr(), y.data_ptr(), N, C, H, W, k, stride, pad, layout, _torch_dtype_code(x),
                                    y_channel_offset, y_channel_stride, _stream()))
    return y


def rtoss_upsample2x(x, y, N, C, H, W, layout=NCHW, y_channel_offset=0, y_channel_stride=0):
    _glue_check(lib.rtoss_upsample2x(x.data_ptr(), y.data_ptr(), N, C, H, W, layout, _torch_dtype_code(x), y_channel_offset,
                                     y_channel_stride, _stream()))
    return y


def rtoss_add_act(a, b, y, act=ACT_NONE):
    _glue_check(lib.rtoss_add_act(a.data_ptr(), b.data_ptr(), y.data_ptr(), a.numel(), _torch_dtype_code(a), act, _stream()))
    return y


def rtoss_fma_plan3x3(N, H, W, stride, layout, io_dtype, Cin, Cout, k, packed_dtype=None):
    """The tiling the FMA path would use for a 3x3 call (host only) -> FmaPlan; raises on an argument error."""
    d = ConvDesc(int(N), int(H), int(W), int(stride), int(layout), int(io_dtype), 0, None, 0, 0, 0, None, 0)
    out = FmaPlan()
    st = lib.rtoss_fma_plan3x3(ctypes.byref(d), int(Cin), int(Cout), int(k), int(io_dtype if packed_dtype is None else packed_dtype),
                               ctypes.byref(out))
    if st != OK:
        raise RtossError(st, status_string(st))
    return out


def rtoss_tensor_plan_of(N, H, W, stride, ksize, Cin, Cout, dtype, sm_count=0, layout=NHWC, residual=False):
    """The tiling the tensor path would use for a call (host only) -> TensorPlan; raises on an argument error."""
    d = ConvDesc(int(N), int(H), int(W), int(stride), int(layout), int(dtype), 0, None, 0, 0, 0, None, 0)
    if residual:
        d.residual_dev = 1   # (only asked whether there is one)
    out = TensorPlan()
    st = lib.rtoss_tensor_plan_of(ctypes.byref(d), int(ksize), int(Cin), int(Cout), int(dtype), int(sm_count), ctypes.byref(out))
    if st != OK:
        raise RtossError(st, status_string(st))
    return out


def rtoss_chain_deps(items):
    """Which earlier items each conv_item(...) entry has to wait for, from the operands' address ranges -> list of masks."""
    arr = (ConvItem * len(items))(*items)
    out = (ctypes.c_uint32 * len(items))()
    st = lib.rtoss_chain_deps(arr, len(items), out)
    if st != OK:
        raise RtossError(st, status_string(st))
    return list(out)


def rtoss_chain_deps_spans(spans):
    """spans: per item (x_lo, x_hi, y_lo, y_hi, r_lo, r_hi) byte ranges -> list of masks (host arithmetic only)."""
    flat = (ctypes.c_uint64 * (6 * len(spans)))(*[int(v) for sp in spans for v in sp])
    out = (ctypes.c_uint32 * len(spans))()
    st = lib.rtoss_chain_deps_spans(flat, len(spans), out)
    if st != OK:
        raise RtossError(st, status_string(st))
    return list(out)


def rtoss_prune_dense_static(w, ksize, masks, k, out=None):
    """Pruned dense weights W (.) mask without any allocation inside the library (the ids live in a fixed
    device array of the library; at most 2^20 kernels).  `out` is a caller-owned tensor like `w`; the one
    created here when it is omitted is the caller's convenience, not the library's doing.  Returns the
    status code together with the tensor so that callers can test for RTOSS_ERR_UNSUPPORTED."""
    import torch
    m = _masks_arr(masks)
    if out is None:
        out = torch.empty_like(w)
    st = lib.rtoss_prune_dense_static(w.data_ptr(), _torch_dtype_code(w), int(w.shape[0]), int(w.shape[1]), int(ksize),
                                      _np_ptr(m), len(m), int(k), out.data_ptr(), _stream())
    return st, out


def _torch_dtype_code(t):
    import torch
    return {torch.float32: F32, torch.bfloat16: BF16, torch.float16: F16}[t.dtype]


def _stream():
    import torch
    return ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)


class Context:
    """Owns an rtoss_ctx on one CUDA device."""

    def __init__(self, device=0):
        h = ctypes.c_void_p()
        st = lib.rtoss_create(int(device), ctypes.byref(h))
        if st != OK:
            raise RtossError(st, "rtoss_create: " + status_string(st) + " (a CUDA device is required)")
        self.h = h
        self.device = device

    def close(self):
        if self.h:
            lib.rtoss_destroy(self.h)
            self.h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def _check(self, st):
        if st != OK:
            raise RtossError(st, status_string(st) + " -- " + lib.rtoss_last_error(self.h).decode())

    # -- the four calls of the hot path ------------------------------------------------
    def rtoss_select_patterns(self, w, ksize, masks, k, pid=None):
        """w: CUDA tensor [Cout,Cin,3,3] or [Cout,Cin(,1,1)] -> uint8 CUDA tensor of pattern ids."""
        import torch
        Cout, Cin = int(w.shape[0]), int(w.shape[1])
        m = _masks_arr(masks)
        n = Cout * Cin if ksize == 3 else (Cout * Cin) // 9
        if pid is None:
            pid = torch.empty(max(n, 1), dtype=torch.uint8, device=w.device)
        self._check(lib.rtoss_select_patterns(self.h, w.data_ptr(), _torch_dtype_code(w), Cout, Cin, int(ksize),
                                              _np_ptr(m), len(m), int(k), pid.data_ptr(), _stream()))
        return pid[:n]

    def rtoss_select_patterns_shared(self, w, masks, k, filter_block, channel_block, pid=None):
        """w: CUDA tensor [Cout,Cin,3,3] -> uint8 ids [Cout*Cin], one pattern per block of filters x channels."""
        import torch
        Cout, Cin = int(w.shape[0]), int(w.shape[1])
        m = _masks_arr(masks)
        if pid is None:
            pid = torch.empty(Cout * Cin, dtype=torch.uint8, device=w.device)
        self._check(lib.rtoss_select_patterns_shared(self.h, w.data_ptr(), _torch_dtype_code(w), Cout, Cin, int(filter_block),
                                                     int(channel_block), _np_ptr(m), len(m), int(k), pid.data_ptr(), _stream()))
        return pid

    def rtoss_pattern_usage(self, kernels, masks, k):
        """kernels: CUDA tensor [n, 9] (or [n,3,3]) -> numpy uint64 win counts per pattern of the table."""
        import torch
        m = _masks_arr(masks)
        n = kernels.numel() // 9
        scratch = torch.empty(n, dtype=torch.uint8, device=kernels.device)
        counts = torch.zeros(len(m), dtype=torch.int64, device=kernels.device)
        self._check(lib.rtoss_pattern_usage(self.h, kernels.data_ptr(), _torch_dtype_code(kernels), n, _np_ptr(m), len(m),
                                            int(k), scratch.data_ptr(), counts.data_ptr(), _stream()))
        return counts.cpu().numpy().astype(np.uint64)

    def rtoss_pattern_table_derive(self, kernels, k, preset, M):
        """kernels: CUDA tensor [n, 9] -> (kept masks ascending, candidate masks, candidate counts)."""
        import torch
        n = kernels.numel() // 9
        scratch = torch.empty(n, dtype=torch.uint8, device=kernels.device)
        counts_dev = torch.zeros(255, dtype=torch.int64, device=kernels.device)
        top = np.zeros(max(int(M), 1), dtype=np.uint16)
        cand = np.zeros(255, dtype=np.uint16)
        cnt = np.zeros(255, dtype=np.uint64)
        kept, P = ctypes.c_int(0), ctypes.c_int(0)
        self._check(lib.rtoss_pattern_table_derive(self.h, kernels.data_ptr(), _torch_dtype_code(kernels), n, int(k), int(preset),
                                                   int(M), scratch.data_ptr(), counts_dev.data_ptr(), _np_ptr(top),
                                                   ctypes.byref(kept), _np_ptr(cand), _np_ptr(cnt), ctypes.byref(P), _stream()))
        return top[:kept.value].copy(), cand[:P.value].copy(), cnt[:P.value].copy()

    def rtoss_pack(self, w, ksize, masks, k, pid, compute_dtype, into=None):
        """New packed handle, or re-pack `into` (an existing handle of the same layer) without allocating."""
        Cout, Cin = int(w.shape[0]), int(w.shape[1])
        m = _masks_arr(masks)
        h = ctypes.c_void_p(into.h.value) if into is not None else ctypes.c_void_p()
        self._check(lib.rtoss_pack(self.h, w.data_ptr(), _torch_dtype_code(w), Cout, Cin, int(ksize), _np_ptr(m),
                                   len(m), int(k), pid.data_ptr(), int(compute_dtype), ctypes.byref(h), _stream()))
        return into if into is not None else Packed(self, h)

    def rtoss_batch_create(self, items):
        """items: list of dict(w, ksize, masks, k, packed, pid=None, pid_from=-1) -> Batch (whole-model pass)."""
        return Batch(self, items)

    def _desc(self, x_shape_nchw, stride, layout, io_dtype, act, bias, y_off, y_stride, path=PATH_AUTO, residual=None,
              residual_after_act=False):
        N, _, H, W = x_shape_nchw
        return ConvDesc(int(N), int(H), int(W), int(stride), int(layout), int(io_dtype), int(act),
                        bias.data_ptr() if bias is not None else None, int(y_off), int(y_stride), int(path),
                        residual.data_ptr() if residual is not None else None, 1 if residual_after_act else 0)

    def rtoss_device_status(self):
        """Synchronise the device and return the code a timed-out device wait left (0 = none)."""
        code = ctypes.c_int(0)
        st = lib.rtoss_device_status(self.h, ctypes.byref(code))
        if st not in (OK, 7):
            self._check(st)
        return code.value

    def rtoss_conv3x3_pattern(self, packed, x, y, N, H, W, stride=1, layout=NCHW, act=ACT_NONE, bias=None,
                              y_channel_offset=0, y_channel_stride=0, path=PATH_AUTO, residual=None, residual_after_act=False):
        d = self._desc((N, 0, H, W), stride, layout, _torch_dtype_code(x), act, bias, y_channel_offset, y_channel_stride,
                       path, residual, residual_after_act)
        self._check(lib.rtoss_conv3x3_pattern(self.h, packed.h, x.data_ptr(), y.data_ptr(), ctypes.byref(d), _stream()))
        return y

    def rtoss_conv1x1_pattern(self, packed, x, y, N, H, W, stride=1, layout=NCHW, act=ACT_NONE, bias=None,
                              y_channel_offset=0, y_channel_stride=0, path=PATH_AUTO, residual=None, residual_after_act=False):
        d = self._desc((N, 0, H, W), stride, layout, _torch_dtype_code(x), act, bias, y_channel_offset, y_channel_stride,
                       path, residual, residual_after_act)
        self._check(lib.rtoss_conv1x1_pattern(self.h, packed.h, x.data_ptr(), y.data_ptr(), ctypes.byref(d), _stream()))
        return y

    def conv_item(self, packed, x, y, N, H, W, stride=1, layout=NCHW, act=ACT_NONE, bias=None, y_channel_offset=0,
                  y_channel_stride=0, path=PATH_AUTO, residual=None, residual_after_act=False):
        """One entry for rtoss_conv_group (arguments as rtoss_conv3x3_pattern / rtoss_conv1x1_pattern)."""
        d = self._desc((N, 0, H, W), stride, layout, _torch_dtype_code(x), act, bias, y_channel_offset, y_channel_stride,
                       path, residual, residual_after_act)
        return ConvItem(packed.h.value, x.data_ptr(), y.data_ptr(), d)

    def rtoss_conv_group(self, items):
        """items: list of conv_item(...) -> number of kernel launches made."""
        arr = (ConvItem * len(items))(*items)
        n = ctypes.c_int(0)
        self._check(lib.rtoss_conv_group(self.h, arr, len(items), ctypes.byref(n), _stream()))
        return n.value

    def rtoss_conv_chain(self, items, after=None):
        """items: conv_item(...) entries in an order in which they could run one after the other; after: per item the
        bit mask of earlier items it waits for (None: derived from the operands' addresses) -> kernel launches made."""
        arr = (ConvItem * len(items))(*items)
        aft = None if after is None else (ctypes.c_uint32 * len(items))(*[int(a) for a in after])
        n = ctypes.c_int(0)
        self._check(lib.rtoss_conv_chain(self.h, arr, len(items), aft, ctypes.byref(n), _stream()))
        return n.value

    def rtoss_set_wait_limit(self, sm_cycles):
        self._check(lib.rtoss_set_wait_limit(self.h, int(sm_cycles)))

    def rtoss_inject_lost_copy(self):
        self._check(lib.rtoss_inject_lost_copy(self.h))

    def rtoss_conv_pattern_host(self, packed, x_host, y_host, N, H, W, stride=1, layout=NCHW, act=ACT_NONE, bias=None,
                                y_channel_offset=0, y_channel_stride=0, path=PATH_AUTO):
        """x_host / y_host: CPU torch tensors (pinned or not); blocks until y_host is written."""
        d = self._desc((N, 0, H, W), stride, layout, _torch_dtype_code(x_host), act, bias, y_channel_offset,
                       y_channel_stride, path)
        self._check(lib.rtoss_conv_pattern_host(self.h, packed.h, x_host.data_ptr(), y_host.data_ptr(), ctypes.byref(d)))
        return y_host


class Batch:
    """Owns an rtoss_batch: selection + packing of every layer of a model in two launches."""

    def __init__(self, ctx, items):
        self.ctx = ctx
        self._keep = []   # tensors, tables and handles the batch points at
        arr = (BatchItem * max(len(items), 1))()
        for i, it in enumerate(items):
            w, m = it["w"], _masks_arr(it["masks"])
            pid = it.get("pid")
            self._keep.append((w, m, pid, it["packed"]))
            arr[i] = BatchItem(w.data_ptr(), _torch_dtype_code(w), int(w.shape[0]), int(w.shape[1]), int(it["ksize"]),
                               m.ctypes.data, len(m), int(it["k"]),
                               pid.data_ptr() if pid is not None and pid.numel() else None, it["packed"].h,
                               int(it.get("pid_from", -1)))
        self.h = ctypes.c_void_p()
        ctx._check(lib.rtoss_batch_create(ctx.h, arr, len(items), ctypes.byref(self.h)))

    def rtoss_batch_select_pack(self):
        self.ctx._check(lib.rtoss_batch_select_pack(self.ctx.h, self.h, _stream()))

    def close(self):
        if self.h:
            lib.rtoss_batch_destroy(self.h)
            self.h = ctypes.c_void_p()


class Packed:
    """Owns an rtoss_packed handle."""

    def __init__(self, ctx, h):
        self.ctx = ctx
        self.h = h
        info = PackedInfo()
        lib.rtoss_packed_info_get(h, ctypes.byref(info))
        self.info = info

    def export(self):
        """-> dict of numpy arrays: pid, val (uint16 bits for 16-bit types, float32 else), perm, bucket_off."""
        i = self.info
        pid = np.zeros(max(i.n_kernels, 1), dtype=np.uint8)
        val = np.zeros(max(i.n_values, 1), dtype=np.float32 if i.dtype == F32 else np.uint16)
        perm = np.zeros(max(i.Cin * i.Cout, 1), dtype=np.uint32)
        off = np.zeros(max(i.Cin * (i.P + 1), 1), dtype=np.uint32)
        self.ctx._check(lib.rtoss_packed_export(self.ctx.h, self.h, _np_ptr(pid), _np_ptr(val), _np_ptr(perm),
                                                _np_ptr(off), _stream()))
        out = dict(pid=pid[:i.n_kernels], val=val[:i.n_values])
        if i.ksize == 3:
            out["perm"] = perm[:i.Cin * i.Cout]
            out["bucket_off"] = off[:i.Cin * (i.P + 1)]
        return out

    def to_dense(self):
        import torch
        i = self.info
        td = {F32: torch.float32, BF16: torch.bfloat16, F16: torch.float16}[i.dtype]
        shape = (i.Cout, i.Cin, 3, 3) if i.ksize == 3 else (i.Cout, i.Cin)
        out = torch.empty(shape, dtype=td, device="cuda:%d" % self.ctx.device)
        self.ctx._check(lib.rtoss_packed_to_dense(self.ctx.h, self.h, out.data_ptr(), _stream()))
        return out

    def close(self):
        if self.h:
            lib.rtoss_packed_destroy(self.h)
            self.h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass
