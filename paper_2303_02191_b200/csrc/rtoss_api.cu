// C-ABI entry points of librtoss that touch the device: argument validation,
// handle lifetimes, kernel launches.  See include/rtoss.h for the contract.
#include <cuda_runtime.h>

#include <cstdio>
#include <cstring>
#include <vector>
#include <new>

#include "rtoss.h"
#include "rtoss_internal.h"

namespace {

void set_err(rtoss_ctx* ctx, const char* what, const char* detail) {
    if (ctx) snprintf(ctx->err, sizeof(ctx->err), "%s%s%s", what, detail ? ": " : "", detail ? detail : "");
}

rtoss_status cuda_fail(rtoss_ctx* ctx, const char* where, int e) {
    set_err(ctx, where, cudaGetErrorString((cudaError_t)e));
    return RTOSS_ERR_CUDA;
}

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }
bool dtype_ok(int d) { return d == RTOSS_F32 || d == RTOSS_BF16 || d == RTOSS_F16; }

MaskTable make_table(const uint16_t* masks, int P) {
    MaskTable t;
    memset(&t, 0, sizeof(t));
    memcpy(t.m, masks, sizeof(uint16_t) * (size_t)P);
    return t;
}

rtoss_status check_layer(rtoss_ctx* ctx, int Cout, int Cin, int ksize) {
    if (Cout < 1 || Cin < 1 || (ksize != 1 && ksize != 3)) {
        set_err(ctx, "layer shape", "need Cout, Cin >= 1 and ksize 1 or 3");
        return RTOSS_ERR_INVALID_ARG;
    }
    if ((int64_t)Cout * Cin > (int64_t)1 << 28) {
        set_err(ctx, "layer shape", "Cout*Cin above 2^28");
        return RTOSS_ERR_UNSUPPORTED;
    }
    return RTOSS_OK;
}

rtoss_status check_conv(rtoss_ctx* ctx, const rtoss_packed* p, const void* x, void* y, const rtoss_conv_desc* d,
                        int ksize, bool device_ptrs) {
    if (!ctx) return RTOSS_ERR_INVALID_ARG;
    if (!p || !x || !y || !d) {
        set_err(ctx, "conv", "null argument");
        return RTOSS_ERR_INVALID_ARG;
    }
    if (p->ksize != ksize) {
        set_err(ctx, "conv", "packed handle has the other kernel size");
        return RTOSS_ERR_INVALID_ARG;
    }
    if (p->device != ctx->device) {
        set_err(ctx, "conv", "packed handle lives on another device");
        return RTOSS_ERR_INVALID_ARG;
    }
    if (d->N < 1 || d->H < 1 || d->W < 1 || (d->stride != 1 && d->stride != 2) || !dtype_ok(d->io_dtype) ||
        (d->layout != RTOSS_NCHW && d->layout != RTOSS_NHWC) ||
        (d->act != RTOSS_ACT_NONE && d->act != RTOSS_ACT_RELU && d->act != RTOSS_ACT_SILU) ||
        (d->path != RTOSS_PATH_AUTO && d->path != RTOSS_PATH_FMA && d->path != RTOSS_PATH_TENSOR)) {
        set_err(ctx, "conv", "bad descriptor (N,H,W >= 1; stride 1|2; dtype; layout; act; path)");
        return RTOSS_ERR_INVALID_ARG;
    }
    const int cs = d->y_channel_stride ? d->y_channel_stride : p->Cout;
    if (d->y_channel_offset < 0 || cs < d->y_channel_offset + p->Cout) {
        set_err(ctx, "conv", "output channel slice does not fit y_channel_stride");
        return RTOSS_ERR_INVALID_ARG;
    }
    if ((int64_t)d->H * d->W > (int64_t)1 << 30) {
        set_err(ctx, "conv", "H*W above 2^30");
        return RTOSS_ERR_UNSUPPORTED;
    }
    if (device_ptrs && (!aligned16(x) || !aligned16(y))) {
        set_err(ctx, "conv", "x and y must be 16-byte aligned");
        return RTOSS_ERR_ALIGNMENT;
    }
    return RTOSS_OK;
}

// Pick the kernel family for one convolution call and launch it.  Returns the CUDA error code of
// the launch; *st is set when the requested path cannot take the call.
int dispatch_conv(rtoss_ctx* ctx, const rtoss_packed* p, const void* x, void* y, const rtoss_conv_desc* d, void* stream,
                  rtoss_status* st) {
    *st = RTOSS_OK;
    const bool tc_ok = d->path != RTOSS_PATH_FMA && rtoss_tc_eligible(p, d, x, y);
    if (d->residual_dev && !tc_ok) {
        set_err(ctx, "conv", "a residual operand is only taken by the tensor path (see rtoss.h)");
        *st = RTOSS_ERR_UNSUPPORTED;
        return 0;
    }
    if (d->path == RTOSS_PATH_TENSOR && !tc_ok) {
        set_err(ctx, "conv", "the tensor path does not take this call (see rtoss.h for its conditions)");
        *st = RTOSS_ERR_UNSUPPORTED;
        return 0;
    }
    if (tc_ok) return rtoss_launch_conv_tc(ctx, p, x, y, d, stream);
    return p->ksize == 3 ? rtoss_launch_conv3x3(ctx, p, x, y, d, stream) : rtoss_launch_conv1x1(ctx, p, x, y, d, stream);
}

}  // namespace

rtoss_device_guard::rtoss_device_guard(int device) : prev(device), switched(false) {
    if (cudaGetDevice(&prev) == cudaSuccess && prev != device) switched = cudaSetDevice(device) == cudaSuccess;
}
rtoss_device_guard::~rtoss_device_guard() {
    if (switched) cudaSetDevice(prev);
}

extern "C" {

rtoss_status rtoss_create(int device, rtoss_ctx** out) {
    if (!out) return RTOSS_ERR_INVALID_ARG;
    *out = nullptr;
    int count = 0;
    cudaError_t e = cudaGetDeviceCount(&count);
    if (e != cudaSuccess || device < 0 || device >= count) return RTOSS_ERR_CUDA;
    cudaDeviceProp prop;
    if (cudaGetDeviceProperties(&prop, device) != cudaSuccess) return RTOSS_ERR_CUDA;
    if (prop.major < 10) return RTOSS_ERR_UNSUPPORTED;  // kernels are built for sm_100a only
    rtoss_ctx* c = new (std::nothrow) rtoss_ctx();
    if (!c) return RTOSS_ERR_ALLOC;
    memset(c, 0, sizeof(*c));
    c->device = device;
    c->sm_count = prop.multiProcessorCount;
    int prev = 0;
    cudaGetDevice(&prev);
    cudaSetDevice(device);
    cudaError_t se = cudaMalloc((void**)&c->dev_status, sizeof(int));
    if (se == cudaSuccess) se = cudaMemset(c->dev_status, 0, sizeof(int));
    const size_t chain_bytes = sizeof(unsigned) * RTOSS_CHAIN_SLOTS * RTOSS_CHAIN_SLOT_WORDS;
    if (se == cudaSuccess) se = cudaMalloc((void**)&c->chain_done, chain_bytes);
    if (se == cudaSuccess) se = cudaMemset(c->chain_done, 0, chain_bytes);
    if (se != cudaSuccess) {
        if (c->dev_status) cudaFree(c->dev_status);
        if (c->chain_done) cudaFree(c->chain_done);
    }
    cudaSetDevice(prev);
    if (se != cudaSuccess) {
        cudaGetLastError();
        delete c;
        return RTOSS_ERR_ALLOC;
    }
    *out = c;
    return RTOSS_OK;
}

void rtoss_destroy(rtoss_ctx* ctx) {
    if (!ctx) return;
    int prev = 0;
    cudaGetDevice(&prev);
    cudaSetDevice(ctx->device);
    if (ctx->h_stream) {
        cudaDeviceSynchronize();
        cudaStreamDestroy((cudaStream_t)ctx->h_stream);
        cudaStreamDestroy((cudaStream_t)ctx->h_stream2);
        cudaStreamDestroy((cudaStream_t)ctx->h_stream3);
        for (int i = 0; i < kHostChunks; ++i) {
            if (ctx->h_ev_in[i]) cudaEventDestroy((cudaEvent_t)ctx->h_ev_in[i]);
            if (ctx->h_ev_run[i]) cudaEventDestroy((cudaEvent_t)ctx->h_ev_run[i]);
        }
    }
    if (ctx->ws_x) cudaFree(ctx->ws_x);
    if (ctx->ws_y) cudaFree(ctx->ws_y);
    if (ctx->dev_status) cudaFree(ctx->dev_status);
    if (ctx->chain_done) cudaFree(ctx->chain_done);
    cudaSetDevice(prev);
    delete ctx;
}

const char* rtoss_last_error(const rtoss_ctx* ctx) { return ctx ? ctx->err : ""; }

rtoss_status rtoss_select_patterns(rtoss_ctx* ctx, const void* w_dev, rtoss_dtype w_dtype, int Cout, int Cin, int ksize,
                                   const uint16_t* masks_host, int P, int k, uint8_t* pid_dev, void* cuda_stream) {
    if (!ctx) return RTOSS_ERR_INVALID_ARG;
    const bool none_sel = ksize == 1 && (int64_t)Cout * Cin < 9;  // no full run of nine: nothing to write
    if (!w_dev || (!pid_dev && !none_sel) || !masks_host || !dtype_ok(w_dtype)) {
        set_err(ctx, "select", "null argument or bad dtype");
        return RTOSS_ERR_INVALID_ARG;
    }
    rtoss_status st = check_layer(ctx, Cout, Cin, ksize);
    if (st != RTOSS_OK) return st;
    if (!rtoss_table_ok(masks_host, P, k)) {
        set_err(ctx, "select", "pattern table invalid");
        return RTOSS_ERR_BAD_PATTERN_TABLE;
    }
    if (!aligned16(w_dev)) {
        set_err(ctx, "select", "weights must be 16-byte aligned");
        return RTOSS_ERR_ALIGNMENT;
    }
    const int64_t n = ksize == 3 ? (int64_t)Cout * Cin : ((int64_t)Cout * Cin) / 9;
    rtoss_device_guard on_device(ctx->device);   // the caller's current device comes back when the call returns
    int e = rtoss_launch_select(w_dev, w_dtype, n, make_table(masks_host, P), P, pid_dev, cuda_stream);
    return e ? cuda_fail(ctx, "select launch", e) : RTOSS_OK;
}

rtoss_status rtoss_select_patterns_shared(rtoss_ctx* ctx, const void* w_dev, rtoss_dtype w_dtype, int Cout, int Cin,
                                          int filter_block, int channel_block, const uint16_t* masks_host, int P, int k,
                                          uint8_t* pid_dev, void* cuda_stream) {
    if (!ctx) return RTOSS_ERR_INVALID_ARG;
    if (!w_dev || !pid_dev || !masks_host || !dtype_ok(w_dtype)) {
        set_err(ctx, "select shared", "null argument or bad dtype");
        return RTOSS_ERR_INVALID_ARG;
    }
    rtoss_status st = check_layer(ctx, Cout, Cin, 3);
    if (st != RTOSS_OK) return st;
    if (filter_block < 1 || filter_block > 256 || channel_block < 1) {
        set_err(ctx, "select shared", "filter_block must be 1..256, channel_block at least 1");
        return RTOSS_ERR_INVALID_ARG;
    }
    if (!rtoss_table_ok(masks_host, P, k)) {
        set_err(ctx, "select shared", "pattern table invalid");
        return RTOSS_ERR_BAD_PATTERN_TABLE;
    }
    if (!aligned16(w_dev)) {
        set_err(ctx, "select shared", "weights must be 16-byte aligned");
        return RTOSS_ERR_ALIGNMENT;
    }
    rtoss_device_guard on_device(ctx->device);
    int e = rtoss_launch_select_shared(w_dev, w_dtype, Cout, Cin, filter_block, channel_block, make_table(masks_host, P), P,
                                       pid_dev, cuda_stream);
    return e ? cuda_fail(ctx, "select shared launch", e) : RTOSS_OK;
}

rtoss_status rtoss_pack(rtoss_ctx* ctx, const void* w_dev, rtoss_dtype w_dtype, int Cout, int Cin, int ksize,
                        const uint16_t* masks_host, int P, int k, const uint8_t* pid_dev, rtoss_dtype compute_dtype,
                        rtoss_packed** out, void* cuda_stream) {
    if (!ctx) return RTOSS_ERR_INVALID_ARG;
    const bool none_sel = ksize == 1 && (int64_t)Cout * Cin < 9;  // no full run of nine: pid may be NULL
    if (!w_dev || (!pid_dev && !none_sel) || !masks_host || !out || !dtype_ok(w_dtype) || !dtype_ok(compute_dtype)) {
        set_err(ctx, "pack", "null argument or bad dtype");
        return RTOSS_ERR_INVALID_ARG;
    }
    rtoss_status st = check_layer(ctx, Cout, Cin, ksize);
    if (st != RTOSS_OK) return st;
    if (!rtoss_table_ok(masks_host, P, k)) {
        set_err(ctx, "pack", "pattern table invalid");
        return RTOSS_ERR_BAD_PATTERN_TABLE;
    }
    if (!aligned16(w_dev)) {
        set_err(ctx, "pack", "weights must be 16-byte aligned");
        return RTOSS_ERR_ALIGNMENT;
    }
    rtoss_device_guard on_device(ctx->device);   // the caller's current device comes back when the call returns
    cudaStream_t s = (cudaStream_t)cuda_stream;
    cudaError_t e = cudaSuccess;
    rtoss_packed* p = *out;
    const bool reuse = p != nullptr;
    bool masks_changed = true;
    if (reuse) {
        // re-pack into an existing handle (e.g. after another pruning iteration): same layer, no allocation
        if (p->device != ctx->device || p->Cout != Cout || p->Cin != Cin || p->ksize != ksize || p->P != P || p->k != k ||
            p->dtype != compute_dtype) {
            set_err(ctx, "pack", "existing handle describes another layer, table size or dtype");
            return RTOSS_ERR_INVALID_ARG;
        }
        masks_changed = memcmp(p->masks, masks_host, sizeof(uint16_t) * (size_t)P) != 0;
        if (masks_changed) {
            memset(p->masks, 0, sizeof(p->masks));
            memcpy(p->masks, masks_host, sizeof(uint16_t) * (size_t)P);
        }
    } else {
        p = new (std::nothrow) rtoss_packed();
        if (!p) return RTOSS_ERR_ALLOC;
        memset(p, 0, sizeof(*p));
        p->device = ctx->device;
        p->Cout = Cout;
        p->Cin = Cin;
        p->ksize = ksize;
        p->P = P;
        p->k = k;
        p->dtype = compute_dtype;
        p->n_kernels = ksize == 3 ? (int64_t)Cout * Cin : ((int64_t)Cout * Cin) / 9;
        memcpy(p->masks, masks_host, sizeof(uint16_t) * (size_t)P);
        const size_t nk = (size_t)(p->n_kernels > 0 ? p->n_kernels : 1);
        e = cudaMalloc((void**)&p->pid, nk);
        if (e == cudaSuccess) e = cudaMalloc(&p->val, nk * (size_t)k * rtoss_dtype_size(compute_dtype));
        if (e == cudaSuccess) e = cudaMalloc((void**)&p->masks_dev, sizeof(uint16_t) * 256);
        if (e == cudaSuccess && ksize == 3) {
            e = cudaMalloc((void**)&p->perm, sizeof(uint32_t) * (size_t)Cin * Cout);
            if (e == cudaSuccess) e = cudaMalloc((void**)&p->bucket_off, sizeof(uint32_t) * (size_t)Cin * (P + 1));
        }
        if (e == cudaSuccess && rtoss_tc_weights_eligible(p)) {
            // dense-expanded weights of the tensor path; zeroed once: the trailing Cout*Cin mod 9 weights of a 1x1
            // layer are pruned for good and no later pack writes them
            const size_t wtc_bytes = (size_t)(ksize == 3 ? 9 : 1) * rtoss_wtc_layout_of(Cout, ksize).rows * Cin *
                                     rtoss_dtype_size(compute_dtype) * (compute_dtype == RTOSS_F32 ? 2 : 1);   // fp32: heads + remainders
            e = cudaMalloc(&p->wtc, wtc_bytes);
            if (e == cudaSuccess) e = cudaMemsetAsync(p->wtc, 0, wtc_bytes, s);
            if (e == cudaSuccess && ksize == 3) {
                p->issue_n = rtoss_issue_words(Cout, Cin, ksize, compute_dtype);
                e = cudaMalloc((void**)&p->issue, sizeof(unsigned long long) * (size_t)p->issue_n);
            }
        }
        if (e != cudaSuccess) {
            cudaGetLastError();
            rtoss_packed_destroy(p);
            set_err(ctx, "pack", "device allocation failed");
            return RTOSS_ERR_ALLOC;
        }
    }
    int le = 0;
    // the mask table is copied from the handle's own (pageable) storage: the copy is staged before return
    if (masks_changed) e = cudaMemcpyAsync(p->masks_dev, p->masks, sizeof(uint16_t) * 256, cudaMemcpyHostToDevice, s);
    if (e == cudaSuccess)  // also writes the handle's own copy of the ids and the tensor path's dense-expanded weights
        le = rtoss_launch_pack_values(w_dev, w_dtype, p->n_kernels, make_table(masks_host, P), pid_dev, k, p->val,
                                      compute_dtype, p->pid, p->wtc, ksize, Cout, Cin, cuda_stream);
    // the ordering pass also gathers which (tap, channel slab) pairs of every filter tile hold kept weights; its words start at zero
    if (e == cudaSuccess && !le && p->issue) e = cudaMemsetAsync(p->issue, 0, sizeof(unsigned long long) * (size_t)p->issue_n, s);
    if (e == cudaSuccess && !le && ksize == 3)
        le = rtoss_launch_pack_order(pid_dev, Cout, Cin, P, p->perm, p->bucket_off, p->masks_dev, p->issue,
                                     rtoss_issue_cb_log2(compute_dtype), cuda_stream);
    if (e != cudaSuccess || le) {
        rtoss_status r = cuda_fail(ctx, "pack launch", e != cudaSuccess ? (int)e : le);
        if (!reuse) rtoss_packed_destroy(p);
        return r;
    }
    *out = p;
    return RTOSS_OK;
}

rtoss_status rtoss_pattern_usage(rtoss_ctx* ctx, const void* kernels_dev, rtoss_dtype dtype, int64_t n_kernels,
                                 const uint16_t* masks_host, int P, int k, uint8_t* pid_scratch_dev, uint64_t* counts_dev,
                                 void* cuda_stream) {
    if (!ctx) return RTOSS_ERR_INVALID_ARG;
    if (!kernels_dev || !masks_host || !pid_scratch_dev || !counts_dev || n_kernels < 1 || !dtype_ok(dtype)) {
        set_err(ctx, "pattern usage", "null argument, bad dtype or no kernels");
        return RTOSS_ERR_INVALID_ARG;
    }
    if (!rtoss_table_ok(masks_host, P, k)) {
        set_err(ctx, "pattern usage", "pattern table invalid");
        return RTOSS_ERR_BAD_PATTERN_TABLE;
    }
    if (!aligned16(kernels_dev)) {
        set_err(ctx, "pattern usage", "kernels must be 16-byte aligned");
        return RTOSS_ERR_ALIGNMENT;
    }
    rtoss_device_guard on_device(ctx->device);   // the caller's current device comes back when the call returns
    cudaStream_t s = (cudaStream_t)cuda_stream;
    cudaError_t e = cudaMemsetAsync(counts_dev, 0, sizeof(uint64_t) * (size_t)P, s);
    if (e != cudaSuccess) return cuda_fail(ctx, "pattern usage", (int)e);
    int le = rtoss_launch_select(kernels_dev, dtype, n_kernels, make_table(masks_host, P), P, pid_scratch_dev, cuda_stream);
    if (!le) le = rtoss_launch_pid_histogram(pid_scratch_dev, n_kernels, P, reinterpret_cast<unsigned long long*>(counts_dev), cuda_stream);
    return le ? cuda_fail(ctx, "pattern usage launch", le) : RTOSS_OK;
}

rtoss_status rtoss_pattern_table_derive(rtoss_ctx* ctx, const void* kernels_dev, rtoss_dtype dtype, int64_t n_kernels,
                                        int k, rtoss_preset preset, int M, uint8_t* pid_scratch_dev, uint64_t* counts_dev,
                                        uint16_t* top_masks_host, int* M_kept, uint16_t* cand_masks_host,
                                        uint64_t* cand_counts_host, int* P_candidates, void* cuda_stream) {
    if (!ctx) return RTOSS_ERR_INVALID_ARG;
    if (!top_masks_host || !M_kept || M < 1 || (preset != RTOSS_PRESET_ALL && preset != RTOSS_PRESET_CONN4)) {
        set_err(ctx, "pattern table derive", "null argument, M < 1 or a preset that is not a candidate family");
        return RTOSS_ERR_INVALID_ARG;
    }
    uint16_t cand[255];
    int P = 255;
    rtoss_status st = rtoss_pattern_preset(k, preset, cand, &P);
    if (st != RTOSS_OK) {
        set_err(ctx, "pattern table derive", "bad k for the preset");
        return st;
    }
    st = rtoss_pattern_usage(ctx, kernels_dev, dtype, n_kernels, cand, P, k, pid_scratch_dev, counts_dev, cuda_stream);
    if (st != RTOSS_OK) return st;
    uint64_t counts[255];
    cudaStream_t s = (cudaStream_t)cuda_stream;
    cudaError_t e = cudaMemcpyAsync(counts, counts_dev, sizeof(uint64_t) * (size_t)P, cudaMemcpyDeviceToHost, s);
    if (e == cudaSuccess) e = cudaStreamSynchronize(s);
    if (e != cudaSuccess) return cuda_fail(ctx, "pattern table derive", (int)e);
    const int keep = M < P ? M : P;
    st = rtoss_pattern_rank(cand, counts, P, k, keep, top_masks_host, nullptr);
    if (st != RTOSS_OK) return st;
    *M_kept = keep;
    if (P_candidates) *P_candidates = P;
    if (cand_masks_host) memcpy(cand_masks_host, cand, sizeof(uint16_t) * (size_t)P);
    if (cand_counts_host) memcpy(cand_counts_host, counts, sizeof(uint64_t) * (size_t)P);
    return RTOSS_OK;
}

rtoss_status rtoss_packed_info_get(const rtoss_packed* p, rtoss_packed_info* info) {
    if (!p || !info) return RTOSS_ERR_INVALID_ARG;
    info->Cout = p->Cout;
    info->Cin = p->Cin;
    info->ksize = p->ksize;
    info->P = p->P;
    info->k = p->k;
    info->dtype = p->dtype;
    info->n_kernels = p->n_kernels;
    info->n_values = p->n_kernels * p->k;
    return RTOSS_OK;
}

rtoss_status rtoss_packed_export(rtoss_ctx* ctx, const rtoss_packed* p, uint8_t* pid_host, void* val_host,
                                 uint32_t* perm_host, uint32_t* bucket_off_host, void* cuda_stream) {
    if (!ctx || !p) return RTOSS_ERR_INVALID_ARG;
    rtoss_device_guard on_device(p->device);   // the caller's current device comes back when the call returns
    cudaStream_t s = (cudaStream_t)cuda_stream;
    cudaError_t e = cudaSuccess;
    if (pid_host && p->n_kernels > 0) e = cudaMemcpyAsync(pid_host, p->pid, (size_t)p->n_kernels, cudaMemcpyDeviceToHost, s);
    if (e == cudaSuccess && val_host && p->n_kernels > 0)
        e = cudaMemcpyAsync(val_host, p->val, (size_t)p->n_kernels * p->k * rtoss_dtype_size(p->dtype),
                            cudaMemcpyDeviceToHost, s);
    if (e == cudaSuccess && p->ksize == 3 && perm_host)
        e = cudaMemcpyAsync(perm_host, p->perm, sizeof(uint32_t) * (size_t)p->Cin * p->Cout, cudaMemcpyDeviceToHost, s);
    if (e == cudaSuccess && p->ksize == 3 && bucket_off_host)
        e = cudaMemcpyAsync(bucket_off_host, p->bucket_off, sizeof(uint32_t) * (size_t)p->Cin * (p->P + 1),
                            cudaMemcpyDeviceToHost, s);
    if (e == cudaSuccess) e = cudaStreamSynchronize(s);
    return e == cudaSuccess ? RTOSS_OK : cuda_fail(ctx, "packed export", (int)e);
}

rtoss_status rtoss_packed_to_dense(rtoss_ctx* ctx, const rtoss_packed* p, void* w_masked_dev, void* cuda_stream) {
    if (!ctx || !p || !w_masked_dev) return RTOSS_ERR_INVALID_ARG;
    rtoss_device_guard on_device(p->device);   // the caller's current device comes back when the call returns
    int e = rtoss_launch_to_dense(p, w_masked_dev, cuda_stream);
    return e ? cuda_fail(ctx, "to_dense launch", e) : RTOSS_OK;
}

void rtoss_packed_destroy(rtoss_packed* p) {
    if (!p) return;
    int prev = 0;
    cudaGetDevice(&prev);
    cudaSetDevice(p->device);
    cudaDeviceSynchronize();
    if (p->pid) cudaFree(p->pid);
    if (p->val) cudaFree(p->val);
    if (p->perm) cudaFree(p->perm);
    if (p->bucket_off) cudaFree(p->bucket_off);
    if (p->masks_dev) cudaFree(p->masks_dev);
    if (p->wtc) cudaFree(p->wtc);
    if (p->issue) cudaFree(p->issue);
    cudaSetDevice(prev);
    delete p;
}

rtoss_status rtoss_conv3x3_pattern(rtoss_ctx* ctx, const rtoss_packed* p, const void* x_dev, void* y_dev,
                                   const rtoss_conv_desc* desc, void* cuda_stream) {
    rtoss_status st = check_conv(ctx, p, x_dev, y_dev, desc, 3, true);
    if (st != RTOSS_OK) return st;
    rtoss_device_guard on_device(ctx->device);   // the caller's current device comes back when the call returns
    int e = dispatch_conv(ctx, p, x_dev, y_dev, desc, cuda_stream, &st);
    if (st != RTOSS_OK) return st;
    return e ? cuda_fail(ctx, "conv3x3 launch", e) : RTOSS_OK;
}

rtoss_status rtoss_conv1x1_pattern(rtoss_ctx* ctx, const rtoss_packed* p, const void* x_dev, void* y_dev,
                                   const rtoss_conv_desc* desc, void* cuda_stream) {
    rtoss_status st = check_conv(ctx, p, x_dev, y_dev, desc, 1, true);
    if (st != RTOSS_OK) return st;
    rtoss_device_guard on_device(ctx->device);   // the caller's current device comes back when the call returns
    int e = dispatch_conv(ctx, p, x_dev, y_dev, desc, cuda_stream, &st);
    if (st != RTOSS_OK) return st;
    return e ? cuda_fail(ctx, "conv1x1 launch", e) : RTOSS_OK;
}

rtoss_status rtoss_conv_group(rtoss_ctx* ctx, const rtoss_conv_item* items, int n, int* launches, void* cuda_stream) {
    if (!ctx) return RTOSS_ERR_INVALID_ARG;
    if (launches) *launches = 0;
    if (!items || n < 1) {
        set_err(ctx, "conv group", "null argument or no items");
        return RTOSS_ERR_INVALID_ARG;
    }
    for (int i = 0; i < n; ++i) {
        if (!items[i].packed) {
            set_err(ctx, "conv group", "item without a packed handle");
            return RTOSS_ERR_INVALID_ARG;
        }
        rtoss_status st = check_conv(ctx, items[i].packed, items[i].x_dev, items[i].y_dev, &items[i].desc, items[i].packed->ksize, true);
        if (st != RTOSS_OK) return st;
    }
    rtoss_device_guard on_device(ctx->device);
    // Items that can share a launch are collected class by class (kernel size, data type, stride for 3x3; tensor path,
    // filters on M), at most twenty to a launch; whatever is left over, or declined by the launcher, runs as single calls.
    std::vector<char> done((size_t)n, 0);
    int count = 0;
    for (int i = 0; i < n; ++i) {
        if (done[(size_t)i]) continue;
        const rtoss_packed* ps[32];
        const void* xs[32];
        void* ys[32];
        const rtoss_conv_desc* ds[32];
        int idx[32], m = 0;
        const int m_max = rtoss_tc_max_problems();
        for (int j = i; j < n && m < m_max; ++j) {
            if (done[(size_t)j]) continue;
            const rtoss_conv_item& a = items[j];
            const rtoss_conv_item& b = items[i];
            if (a.desc.path == RTOSS_PATH_FMA || !rtoss_tc_groupable(a.packed, &a.desc, a.x_dev, a.y_dev)) continue;
            if (a.packed->ksize != b.packed->ksize || a.packed->dtype != b.packed->dtype) continue;
            if (a.packed->ksize == 3 && a.desc.stride != b.desc.stride) continue;
            ps[m] = a.packed, xs[m] = a.x_dev, ys[m] = a.y_dev, ds[m] = &a.desc, idx[m] = j;
            ++m;
        }
        if (m >= 2 && items[i].desc.path != RTOSS_PATH_FMA) {
            const int e = rtoss_launch_conv_tc_group(ctx, m, ps, xs, ys, ds, cuda_stream);
            if (e == 0) {
                for (int q = 0; q < m; ++q) done[(size_t)idx[q]] = 1;
                ++count;
                continue;
            }
            if (e > 0) return cuda_fail(ctx, "conv group launch", e);
        }
        rtoss_status st = RTOSS_OK;
        const int e = dispatch_conv(ctx, items[i].packed, items[i].x_dev, items[i].y_dev, &items[i].desc, cuda_stream, &st);
        if (st != RTOSS_OK) return st;
        if (e) return cuda_fail(ctx, "conv launch", e);
        done[(size_t)i] = 1;
        ++count;
    }
    if (launches) *launches = count;
    return RTOSS_OK;
}

namespace {

// Bytes a convolution call touches: [lo, hi) of its input, its output (the whole pixel pitch where it writes a
// channel slice) and its residual operand.
struct Span {
    uintptr_t lo, hi;
};
inline bool overlap(const Span& a, const Span& b) { return a.lo < b.hi && b.lo < a.hi && a.lo != a.hi && b.lo != b.hi; }
void spans_of(const rtoss_conv_item& it, Span* x, Span* y, Span* r) {
    const rtoss_packed* p = it.packed;
    const rtoss_conv_desc& d = it.desc;
    const size_t es = rtoss_dtype_size(d.io_dtype);
    const int S = d.stride > 0 ? d.stride : 1;
    const size_t Ho = (size_t)((d.H - 1) / S + 1), Wo = (size_t)((d.W - 1) / S + 1);
    const size_t pitch = d.y_channel_stride ? (size_t)d.y_channel_stride : (size_t)p->Cout;
    x->lo = reinterpret_cast<uintptr_t>(it.x_dev);
    x->hi = x->lo + (size_t)d.N * d.H * d.W * p->Cin * es;
    // (a call that writes a channel slice is given the buffer's base: the span is the whole buffer)
    y->lo = reinterpret_cast<uintptr_t>(it.y_dev);
    y->hi = y->lo + (size_t)d.N * Ho * Wo * pitch * es;
    r->lo = reinterpret_cast<uintptr_t>(d.residual_dev);
    r->hi = d.residual_dev ? r->lo + (size_t)d.N * Ho * Wo * pitch * es : r->lo;
}

}  // namespace

rtoss_status rtoss_chain_deps(const rtoss_conv_item* items, int n, uint32_t* after) {
    if (!items || !after || n < 1 || n > 32) return RTOSS_ERR_INVALID_ARG;
    uint64_t spans[32 * 6];
    for (int i = 0; i < n; ++i) {
        if (!items[i].packed) return RTOSS_ERR_INVALID_ARG;
        Span x, y, r;
        spans_of(items[i], &x, &y, &r);
        uint64_t* q = spans + 6 * i;
        q[0] = x.lo, q[1] = x.hi, q[2] = y.lo, q[3] = y.hi, q[4] = r.lo, q[5] = r.hi;
    }
    return rtoss_chain_deps_spans(spans, n, after);
}

rtoss_status rtoss_chain_deps_spans(const uint64_t* spans, int n, uint32_t* after) {
    if (!spans || !after || n < 1 || n > 32) return RTOSS_ERR_INVALID_ARG;
    Span x[32], y[32], r[32];
    for (int i = 0; i < n; ++i) {
        const uint64_t* q = spans + 6 * i;
        if (q[0] > q[1] || q[2] > q[3] || q[4] > q[5]) return RTOSS_ERR_INVALID_ARG;
        x[i] = Span{(uintptr_t)q[0], (uintptr_t)q[1]};
        y[i] = Span{(uintptr_t)q[2], (uintptr_t)q[3]};
        r[i] = Span{(uintptr_t)q[4], (uintptr_t)q[5]};
    }
    for (int i = 0; i < n; ++i) {
        after[i] = 0;
        for (int j = 0; j < i; ++j) {
            const bool reads_j = overlap(x[i], y[j]) || overlap(r[i], y[j]);                          // i reads what j writes
            const bool clobbers_j = overlap(y[i], x[j]) || overlap(y[i], r[j]) || overlap(y[i], y[j]);  // i overwrites what j reads or writes
            if (reads_j || clobbers_j) after[i] |= 1u << j;
        }
    }
    return RTOSS_OK;
}

rtoss_status rtoss_conv_chain(rtoss_ctx* ctx, const rtoss_conv_item* items, int n, const uint32_t* after, int* launches,
                              void* cuda_stream) {
    if (!ctx) return RTOSS_ERR_INVALID_ARG;
    if (launches) *launches = 0;
    if (!items || n < 1 || n > 32) {
        set_err(ctx, "conv chain", "null argument, no items or more than 32");
        return RTOSS_ERR_INVALID_ARG;
    }
    for (int i = 0; i < n; ++i) {
        if (!items[i].packed) {
            set_err(ctx, "conv chain", "item without a packed handle");
            return RTOSS_ERR_INVALID_ARG;
        }
        rtoss_status st = check_conv(ctx, items[i].packed, items[i].x_dev, items[i].y_dev, &items[i].desc, items[i].packed->ksize, true);
        if (st != RTOSS_OK) return st;
        if (after && (i == 0 ? after[0] != 0 : (after[i] >> i) != 0)) {
            set_err(ctx, "conv chain", "an item may only be ordered behind earlier items");
            return RTOSS_ERR_INVALID_ARG;
        }
    }
    uint32_t derived[32];
    if (!after) {
        rtoss_chain_deps(items, n, derived);
        after = derived;
    }
    rtoss_device_guard on_device(ctx->device);
    // Maximal runs of consecutive items that can share a launch go out as one kernel each; an item that cannot (FMA
    // path, positions on M) or that is better off alone (few tiles, many channel blocks and nothing to run beside it:
    // a launch of its own cuts it along K over several CTAs, a shared launch never does) goes out on its own between them.  The stream orders the launches, so inside a run
    // only the dependencies on items of the same run have to be carried into the kernel.
    const int m_max = rtoss_tc_max_problems();
    // (an item's level: one more than the highest level it waits for; items of one level run side by side)
    int level[32];
    bool member[32];
    for (int q = 0; q < n; ++q) {
        level[q] = 0;
        for (int j = 0; j < q; ++j)
            if ((after[q] >> j) & 1u) level[q] = level[j] + 1 > level[q] ? level[j] + 1 : level[q];
    }
    long tiles[32], level_tiles[33] = {};
    bool alone[32];
    for (int q = 0; q < n; ++q) {
        const rtoss_conv_item& it = items[q];
        member[q] = it.desc.path != RTOSS_PATH_FMA && rtoss_tc_groupable(it.packed, &it.desc, it.x_dev, it.y_dev);
        tiles[q] = 0;
        alone[q] = member[q] && rtoss_tc_prefers_split(ctx, it.packed, &it.desc, &tiles[q]) && it.desc.path == RTOSS_PATH_AUTO;
        if (member[q]) level_tiles[level[q]] += tiles[q];
    }
    // (better alone, unless the others of its level keep every SM busy for several tiles: its own few, long tiles then
    // hide among theirs)
    for (int q = 0; q < n; ++q)
        if (alone[q] && level_tiles[level[q]] - tiles[q] < 4L * ctx->sm_count) member[q] = false;
    int count = 0, i = 0;
    while (i < n) {
        int m = 0;
        while (i + m < n && m < m_max && member[i + m] && items[i + m].packed->dtype == items[i].packed->dtype) ++m;
        if (m >= 2) {
            const rtoss_packed* ps[32];
            const void* xs[32];
            void* ys[32];
            const rtoss_conv_desc* ds[32];
            uint32_t aft[32];
            for (int q = 0; q < m; ++q) {
                const rtoss_conv_item& it = items[i + q];
                ps[q] = it.packed, xs[q] = it.x_dev, ys[q] = it.y_dev, ds[q] = &it.desc;
                aft[q] = (after[i + q] >> i) & ((1u << q) - 1u);
            }
            const int e = rtoss_launch_conv_tc_chain(ctx, m, ps, xs, ys, ds, aft, cuda_stream);
            if (e > 0) return cuda_fail(ctx, "conv chain launch", e);
            if (e == 0) {
                ++count;
                i += m;
                continue;
            }
        }
        // a single item, or a run the launcher declined: one call per item, in order
        const int single = m >= 2 ? m : 1;
        for (int q = 0; q < single; ++q, ++i) {
            rtoss_status st = RTOSS_OK;
            const int e = dispatch_conv(ctx, items[i].packed, items[i].x_dev, items[i].y_dev, &items[i].desc, cuda_stream, &st);
            if (st != RTOSS_OK) return st;
            if (e) return cuda_fail(ctx, "conv launch", e);
            ++count;
        }
    }
    if (launches) *launches = count;
    return RTOSS_OK;
}

rtoss_status rtoss_set_wait_limit(rtoss_ctx* ctx, long long sm_cycles) {
    if (!ctx || sm_cycles < 1000) return RTOSS_ERR_INVALID_ARG;
    ctx->wait_cycles = sm_cycles;
    return RTOSS_OK;
}

rtoss_status rtoss_inject_lost_copy(rtoss_ctx* ctx) {
    if (!ctx) return RTOSS_ERR_INVALID_ARG;
    ctx->inject_next = 1;
    return RTOSS_OK;
}

rtoss_status rtoss_device_status(rtoss_ctx* ctx, int* code) {
    if (!ctx || !code) return RTOSS_ERR_INVALID_ARG;
    rtoss_device_guard on_device(ctx->device);   // the caller's current device comes back when the call returns
    cudaError_t e = cudaDeviceSynchronize();
    if (e == cudaSuccess) e = cudaMemcpy(code, ctx->dev_status, sizeof(int), cudaMemcpyDeviceToHost);
    if (e != cudaSuccess) return cuda_fail(ctx, "device status", (int)e);
    if (*code != 0) {
        cudaMemset(ctx->dev_status, 0, sizeof(int));
        // a launch that gave up may have left its completion counters half counted
        cudaMemset(ctx->chain_done, 0, sizeof(unsigned) * RTOSS_CHAIN_SLOTS * RTOSS_CHAIN_SLOT_WORDS);
        set_err(ctx, "device status", "a bounded wait in a tensor-path kernel ran out");
        return RTOSS_ERR_TIMEOUT;
    }
    return RTOSS_OK;
}

rtoss_status rtoss_conv_pattern_host(rtoss_ctx* ctx, const rtoss_packed* p, const void* x_host, void* y_host,
                                     const rtoss_conv_desc* desc) {
    if (!ctx || !p) return RTOSS_ERR_INVALID_ARG;
    rtoss_status st = check_conv(ctx, p, x_host, y_host, desc, p->ksize, false);
    if (st != RTOSS_OK) return st;
    if (desc->residual_dev) {
        set_err(ctx, "conv", "the host-buffer entry point takes no residual operand");
        return RTOSS_ERR_UNSUPPORTED;
    }
    rtoss_device_guard on_device(ctx->device);   // the caller's current device comes back when the call returns
    const size_t es = rtoss_dtype_size(desc->io_dtype);
    const int Ho = (desc->H - 1) / desc->stride + 1, Wo = (desc->W - 1) / desc->stride + 1;
    const int cs = desc->y_channel_stride ? desc->y_channel_stride : p->Cout;
    const size_t xb = (size_t)desc->N * p->Cin * desc->H * desc->W * es;
    const size_t yb = (size_t)desc->N * cs * Ho * Wo * es;
    cudaError_t e = cudaSuccess;
    if (!ctx->h_stream) {
        cudaStream_t st3[3] = {nullptr, nullptr, nullptr};
        for (int i = 0; i < 3 && e == cudaSuccess; ++i) e = cudaStreamCreateWithFlags(&st3[i], cudaStreamNonBlocking);
        for (int i = 0; i < kHostChunks && e == cudaSuccess; ++i) {
            cudaEvent_t ev;
            e = cudaEventCreateWithFlags(&ev, cudaEventDisableTiming);
            ctx->h_ev_in[i] = ev;
            if (e == cudaSuccess) e = cudaEventCreateWithFlags(&ev, cudaEventDisableTiming);
            ctx->h_ev_run[i] = ev;
        }
        if (e != cudaSuccess) return cuda_fail(ctx, "host path streams", (int)e);
        ctx->h_stream = st3[0];
        ctx->h_stream2 = st3[1];
        ctx->h_stream3 = st3[2];
    }
    if (ctx->ws_x_bytes < xb) {
        if (ctx->ws_x) cudaFree(ctx->ws_x);
        ctx->ws_x = nullptr;
        ctx->ws_x_bytes = 0;
        if (cudaMalloc(&ctx->ws_x, xb) != cudaSuccess) {
            cudaGetLastError();
            set_err(ctx, "host path", "workspace allocation failed");
            return RTOSS_ERR_ALLOC;
        }
        ctx->ws_x_bytes = xb;
    }
    if (ctx->ws_y_bytes < yb) {
        if (ctx->ws_y) cudaFree(ctx->ws_y);
        ctx->ws_y = nullptr;
        ctx->ws_y_bytes = 0;
        if (cudaMalloc(&ctx->ws_y, yb) != cudaSuccess) {
            cudaGetLastError();
            set_err(ctx, "host path", "workspace allocation failed");
            return RTOSS_ERR_ALLOC;
        }
        ctx->ws_y_bytes = yb;
    }
    // Three streams, the batch cut into image chunks: the copy-in of chunk c+1, the kernel of chunk c and the
    // copy-out of chunk c-1 overlap (PCIe is full duplex), so a call costs about max(copy in, copy out).
    const bool slice = cs != p->Cout;
    const size_t x_img = (size_t)p->Cin * desc->H * desc->W * es, y_img = (size_t)cs * Ho * Wo * es;
    int n_chunks = desc->N < kHostChunks ? desc->N : kHostChunks;
    while (n_chunks > 1 && (xb + yb) / n_chunks < ((size_t)1 << 20)) --n_chunks;  // not below ~1 MB per chunk
    cudaStream_t s_in = (cudaStream_t)ctx->h_stream, s_run = (cudaStream_t)ctx->h_stream2, s_out = (cudaStream_t)ctx->h_stream3;
    rtoss_conv_desc dc = *desc;
    int done = 0;
    for (int c = 0; c < n_chunks && e == cudaSuccess; ++c) {
        const int n_c = (desc->N - done + (n_chunks - c) - 1) / (n_chunks - c);
        char* xd = static_cast<char*>(ctx->ws_x) + (size_t)done * x_img;
        char* yd = static_cast<char*>(ctx->ws_y) + (size_t)done * y_img;
        e = cudaMemcpyAsync(xd, static_cast<const char*>(x_host) + (size_t)done * x_img, (size_t)n_c * x_img,
                            cudaMemcpyHostToDevice, s_in);
        // a channel slice leaves the other channels of y untouched: bring the caller's y over first
        if (e == cudaSuccess && slice)
            e = cudaMemcpyAsync(yd, static_cast<const char*>(y_host) + (size_t)done * y_img, (size_t)n_c * y_img,
                                cudaMemcpyHostToDevice, s_in);
        if (e == cudaSuccess) e = cudaEventRecord((cudaEvent_t)ctx->h_ev_in[c], s_in);
        if (e == cudaSuccess) e = cudaStreamWaitEvent(s_run, (cudaEvent_t)ctx->h_ev_in[c], 0);
        if (e != cudaSuccess) break;
        dc.N = n_c;
        int le = dispatch_conv(ctx, p, xd, yd, &dc, s_run, &st);
        if (st != RTOSS_OK || le) {
            cudaDeviceSynchronize();
            if (st != RTOSS_OK) return st;
            return cuda_fail(ctx, "host path launch", le);
        }
        e = cudaEventRecord((cudaEvent_t)ctx->h_ev_run[c], s_run);
        if (e == cudaSuccess) e = cudaStreamWaitEvent(s_out, (cudaEvent_t)ctx->h_ev_run[c], 0);
        if (e == cudaSuccess)
            e = cudaMemcpyAsync(static_cast<char*>(y_host) + (size_t)done * y_img, yd, (size_t)n_c * y_img,
                                cudaMemcpyDeviceToHost, s_out);
        done += n_c;
    }
    if (e == cudaSuccess) e = cudaStreamSynchronize(s_out);
    if (e != cudaSuccess) {
        cudaDeviceSynchronize();
        return cuda_fail(ctx, "host path", (int)e);
    }
    return RTOSS_OK;
}

}  // extern "C"
