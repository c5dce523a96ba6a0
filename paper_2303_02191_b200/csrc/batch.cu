// Whole-model pruning pass: pattern selection (Algorithm 2; Algorithm 3 for 1x1 layers) and packing of EVERY layer
// of a model in two launches instead of three per layer.  The per-kernel arithmetic is the one of the single-layer
// calls (select_core.cuh), so the results are the same bits.
//
//   batch_select_pack_kernel : one thread per kernel / run of nine, 256 per block step; a block step ("chunk")
//                              belongs to one layer, found through a chunk -> layer table built at plan time.
//                              Writes the pattern id (caller's array and the handle's), the k kept values and the
//                              tensor path's dense-expanded weights.
//   batch_order_kernel       : per (3x3 layer, input channel) the stable order of filters by pattern id, one warp
//                              each, through a task -> layer table.
//
// A layer that inherits its parent's patterns (Section IV.A: children of a group share the parent's kernel
// patterns) evaluates the selection on the PARENT's weights and packs its own with the result; it reads no other
// layer's output, so all layers run in the same launch.
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>

#include <cstdio>
#include <cstring>
#include <new>
#include <vector>

#include "conv_common.cuh"
#include "rtoss_internal.h"
#include "select_core.cuh"

namespace {

constexpr int kChunk = 256;     // kernels per block step
constexpr int kOrderWarps = 4;  // channels per block of the ordering kernel

struct BatchLayer {
    const void* w;      // weights to pack
    const void* w_sel;  // weights the selection reads: w, or the group parent's
    uint8_t* pid_out;   // caller's id array (nullable)
    uint8_t* pid;       // the handle's arrays
    void* val;
    void* wtc;
    uint32_t* perm;
    uint32_t* bucket_off;
    unsigned long long* issue;  // the handle's issue words (tensor path, 3x3), or null
    int issue_n;
    long long n_kernels;
    rtoss_wtc_layout lay;  // layout of wtc
    int Cout, Cin, ksize, P, k;
    int w_dtype, sel_dtype, v_dtype;
    unsigned chunk0;  // first chunk of this layer
    unsigned task0;   // first ordering task (3x3 layers)
    uint16_t masks[256];
};

__device__ __forceinline__ float load_any(const unsigned char* raw, int idx, int dtype) {
    if (dtype == RTOSS_F32) return reinterpret_cast<const float*>(raw)[idx];
    if (dtype == RTOSS_BF16) return __bfloat162float(reinterpret_cast<const __nv_bfloat16*>(raw)[idx]);
    return __half2float(reinterpret_cast<const __half*>(raw)[idx]);
}

// 9*count weights of `count` consecutive kernels starting at kernel `first`, as raw bytes, coalesced; 16 bytes per
// thread where the chunk is whole (a whole chunk is a multiple of 16 bytes and the base is 16-byte aligned).
__device__ __forceinline__ void stage_raw(const void* w, long long first, int count, int esize, unsigned char* smem) {
    const unsigned char* src = reinterpret_cast<const unsigned char*>(w) + (size_t)first * 9 * esize;
    const int bytes = count * 9 * esize;
    if (count == kChunk) {
        const uint4* s4 = reinterpret_cast<const uint4*>(src);
        uint4* d4 = reinterpret_cast<uint4*>(smem);
        for (int i = threadIdx.x; i < bytes / 16; i += kChunk) d4[i] = __ldg(s4 + i);
    } else if (esize == 4) {
        const uint32_t* s1 = reinterpret_cast<const uint32_t*>(src);
        uint32_t* d1 = reinterpret_cast<uint32_t*>(smem);
        for (int i = threadIdx.x; i < bytes / 4; i += kChunk) d1[i] = s1[i];
    } else {
        const uint16_t* s1 = reinterpret_cast<const uint16_t*>(src);
        uint16_t* d1 = reinterpret_cast<uint16_t*>(smem);
        for (int i = threadIdx.x; i < bytes / 2; i += kChunk) d1[i] = s1[i];
    }
}

__global__ void __launch_bounds__(kChunk) batch_select_pack_kernel(const BatchLayer* __restrict__ layers,
                                                                   const uint32_t* __restrict__ chunk_layer,
                                                                   unsigned n_chunks) {
    rtoss_dev::pdl_enter_handle_writer();
    __shared__ __align__(16) unsigned char s_sel[kChunk * 9 * 4];
    __shared__ __align__(16) unsigned char s_own[kChunk * 9 * 4];
    __shared__ uint16_t s_masks[256];
    for (unsigned chunk = blockIdx.x; chunk < n_chunks; chunk += gridDim.x) {
        const BatchLayer& L = layers[chunk_layer[chunk]];
        const long long first = (long long)(chunk - L.chunk0) * kChunk;
        const long long left = L.n_kernels - first;
        const int count = (int)(left < kChunk ? left : kChunk);
        const bool inherits = L.w_sel != L.w;
        // the layer's first chunk clears its issue words: the ordering kernel (next launch) ORs the bits in
        if (chunk == L.chunk0 && L.issue)
            for (int i = threadIdx.x; i < L.issue_n; i += kChunk) L.issue[i] = 0ull;
        __syncthreads();  // the previous step's readers are done
        stage_raw(L.w_sel, first, count, L.sel_dtype == RTOSS_F32 ? 4 : 2, s_sel);
        if (inherits) stage_raw(L.w, first, count, L.w_dtype == RTOSS_F32 ? 4 : 2, s_own);
        if ((int)threadIdx.x < L.P) s_masks[threadIdx.x] = L.masks[threadIdx.x];
        __syncthreads();
        if ((int)threadIdx.x < count) {
            const long long i = first + threadIdx.x;
            float v[9];
#pragma unroll
            for (int t = 0; t < 9; ++t) v[t] = load_any(s_sel, threadIdx.x * 9 + t, L.sel_dtype);
            const int best = rtoss_dev::select_best(v, s_masks, L.P);
            if (L.pid_out) L.pid_out[i] = (uint8_t)best;
            L.pid[i] = (uint8_t)best;
            if (inherits) {
#pragma unroll
                for (int t = 0; t < 9; ++t) v[t] = load_any(s_own, threadIdx.x * 9 + t, L.w_dtype);
            }
            const unsigned m = s_masks[best];
            if (L.v_dtype == RTOSS_F32)
                rtoss_dev::pack_one<float>(v, m, i, L.k, (float*)L.val, (float*)L.wtc, L.ksize, L.Cin, L.lay.rows, L.lay.rep_rows,
                                           L.lay.copies);
            else if (L.v_dtype == RTOSS_BF16)
                rtoss_dev::pack_one<__nv_bfloat16>(v, m, i, L.k, (__nv_bfloat16*)L.val, (__nv_bfloat16*)L.wtc, L.ksize, L.Cin,
                                                   L.lay.rows, L.lay.rep_rows, L.lay.copies);
            else
                rtoss_dev::pack_one<__half>(v, m, i, L.k, (__half*)L.val, (__half*)L.wtc, L.ksize, L.Cin, L.lay.rows, L.lay.rep_rows,
                                            L.lay.copies);
        }
    }
}

__global__ void __launch_bounds__(kOrderWarps * 32) batch_order_kernel(const BatchLayer* __restrict__ layers,
                                                                       const uint32_t* __restrict__ task_layer,
                                                                       unsigned n_tasks) {
    rtoss_dev::pdl_enter_handle_writer();
    __shared__ uint32_t fill_all[kOrderWarps][256];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    for (unsigned task = blockIdx.x * kOrderWarps + warp; task < n_tasks; task += gridDim.x * kOrderWarps) {
        const BatchLayer& L = layers[task_layer[task]];
        rtoss_dev::order_channel(L.pid, L.Cout, L.Cin, L.P, (int)(task - L.task0), L.perm, L.bucket_off, fill_all[warp],
                                 lane, L.masks, L.issue, L.v_dtype == RTOSS_F32 ? 5 : 6);
        __syncwarp();
    }
}

void set_err(rtoss_ctx* ctx, const char* what) {
    if (!ctx) return;
    snprintf(ctx->err, sizeof(ctx->err), "batch: %s", what);
}

}  // namespace

struct rtoss_batch {
    int device;
    int L;
    BatchLayer* layers_dev;
    uint32_t* chunk_layer_dev;
    uint32_t* task_layer_dev;
    unsigned n_chunks, n_tasks;
};

extern "C" {

rtoss_status rtoss_batch_create(rtoss_ctx* ctx, const rtoss_batch_item* items, int L, rtoss_batch** out) {
    if (!ctx) return RTOSS_ERR_INVALID_ARG;
    if (!items || L < 1 || !out) {
        set_err(ctx, "null argument or no layers");
        return RTOSS_ERR_INVALID_ARG;
    }
    *out = nullptr;
    std::vector<BatchLayer> layers((size_t)L);
    std::vector<uint32_t> chunk_layer, task_layer;
    for (int i = 0; i < L; ++i) {
        const rtoss_batch_item& it = items[i];
        rtoss_packed* p = it.packed;
        if (!it.w_dev || !p || !it.masks_host || (int)it.w_dtype < 0 || (int)it.w_dtype > 2) {
            set_err(ctx, "item with a null pointer or bad dtype");
            return RTOSS_ERR_INVALID_ARG;
        }
        if (p->device != ctx->device || p->Cout != it.Cout || p->Cin != it.Cin || p->ksize != it.ksize || p->P != it.P ||
            p->k != it.k) {
            set_err(ctx, "item's packed handle describes another layer, table size or device");
            return RTOSS_ERR_INVALID_ARG;
        }
        if (!rtoss_table_ok(it.masks_host, it.P, it.k)) {
            set_err(ctx, "pattern table invalid");
            return RTOSS_ERR_BAD_PATTERN_TABLE;
        }
        if (reinterpret_cast<uintptr_t>(it.w_dev) & 15) {
            set_err(ctx, "weights must be 16-byte aligned");
            return RTOSS_ERR_ALIGNMENT;
        }
        for (int j = 0; j < i; ++j)
            if (items[j].packed == p) {
                set_err(ctx, "two items share one packed handle");
                return RTOSS_ERR_INVALID_ARG;
            }
        BatchLayer& B = layers[(size_t)i];
        memset(&B, 0, sizeof(B));
        B.w = it.w_dev;
        B.w_sel = it.w_dev;
        B.sel_dtype = B.w_dtype = (int)it.w_dtype;
        if (it.pid_from >= 0) {
            // inherit the patterns of an earlier item: same shape and the same table, so that ids mean the same masks
            if (it.pid_from >= i) {
                set_err(ctx, "pid_from must name an earlier item");
                return RTOSS_ERR_INVALID_ARG;
            }
            const rtoss_batch_item& par = items[it.pid_from];
            if (par.Cout != it.Cout || par.Cin != it.Cin || par.ksize != it.ksize || par.P != it.P || par.k != it.k ||
                memcmp(par.masks_host, it.masks_host, sizeof(uint16_t) * (size_t)it.P) != 0) {
                set_err(ctx, "pid_from names a layer of another shape or pattern table");
                return RTOSS_ERR_INVALID_ARG;
            }
            B.w_sel = layers[(size_t)it.pid_from].w_sel;  // the root of the chain
            B.sel_dtype = layers[(size_t)it.pid_from].sel_dtype;
        } else if (it.pid_from != -1) {
            set_err(ctx, "pid_from must be -1 or the index of an earlier item");
            return RTOSS_ERR_INVALID_ARG;
        }
        B.pid_out = it.pid_dev;
        B.pid = p->pid;
        B.val = p->val;
        B.wtc = p->wtc;
        B.perm = p->perm;
        B.bucket_off = p->bucket_off;
        B.issue = p->issue;
        B.issue_n = p->issue_n;
        B.n_kernels = p->n_kernels;
        B.lay = rtoss_wtc_layout_of(it.Cout, it.ksize);
        B.Cout = it.Cout;
        B.Cin = it.Cin;
        B.ksize = it.ksize;
        B.P = it.P;
        B.k = it.k;
        B.v_dtype = (int)p->dtype;
        memcpy(B.masks, it.masks_host, sizeof(uint16_t) * (size_t)it.P);
        B.chunk0 = (unsigned)chunk_layer.size();
        const long long nc = (p->n_kernels + kChunk - 1) / kChunk;
        if ((long long)chunk_layer.size() + nc > 0x7FFFFFFFLL) {
            set_err(ctx, "model too large for one batch");
            return RTOSS_ERR_UNSUPPORTED;
        }
        chunk_layer.insert(chunk_layer.end(), (size_t)nc, (uint32_t)i);
        B.task0 = (unsigned)task_layer.size();
        if (it.ksize == 3) task_layer.insert(task_layer.end(), (size_t)it.Cin, (uint32_t)i);
    }
    rtoss_batch* b = new (std::nothrow) rtoss_batch();
    if (!b) return RTOSS_ERR_ALLOC;
    memset(b, 0, sizeof(*b));
    b->device = ctx->device;
    b->L = L;
    b->n_chunks = (unsigned)chunk_layer.size();
    b->n_tasks = (unsigned)task_layer.size();
    int prev = 0;
    cudaGetDevice(&prev);
    cudaSetDevice(ctx->device);
    cudaError_t e = cudaMalloc((void**)&b->layers_dev, sizeof(BatchLayer) * (size_t)L);
    if (e == cudaSuccess) e = cudaMalloc((void**)&b->chunk_layer_dev, sizeof(uint32_t) * (chunk_layer.size() + 1));
    if (e == cudaSuccess) e = cudaMalloc((void**)&b->task_layer_dev, sizeof(uint32_t) * (task_layer.size() + 1));
    if (e == cudaSuccess) e = cudaMemcpy(b->layers_dev, layers.data(), sizeof(BatchLayer) * (size_t)L, cudaMemcpyHostToDevice);
    if (e == cudaSuccess && !chunk_layer.empty())
        e = cudaMemcpy(b->chunk_layer_dev, chunk_layer.data(), sizeof(uint32_t) * chunk_layer.size(), cudaMemcpyHostToDevice);
    if (e == cudaSuccess && !task_layer.empty())
        e = cudaMemcpy(b->task_layer_dev, task_layer.data(), sizeof(uint32_t) * task_layer.size(), cudaMemcpyHostToDevice);
    // the handles take the batch's tables (a convolution reads the handle's device copy of the masks)
    for (int i = 0; i < L && e == cudaSuccess; ++i) {
        rtoss_packed* p = items[i].packed;
        if (memcmp(p->masks, items[i].masks_host, sizeof(uint16_t) * (size_t)items[i].P) != 0) {
            memset(p->masks, 0, sizeof(p->masks));
            memcpy(p->masks, items[i].masks_host, sizeof(uint16_t) * (size_t)items[i].P);
            e = cudaMemcpy(p->masks_dev, p->masks, sizeof(uint16_t) * 256, cudaMemcpyHostToDevice);
        }
    }
    cudaSetDevice(prev);
    if (e != cudaSuccess) {
        cudaGetLastError();
        rtoss_batch_destroy(b);
        set_err(ctx, "device allocation or upload failed");
        return RTOSS_ERR_ALLOC;
    }
    *out = b;
    return RTOSS_OK;
}

rtoss_status rtoss_batch_select_pack(rtoss_ctx* ctx, const rtoss_batch* b, void* cuda_stream) {
    if (!ctx) return RTOSS_ERR_INVALID_ARG;
    if (!b || b->device != ctx->device) {
        set_err(ctx, "null batch or batch of another device");
        return RTOSS_ERR_INVALID_ARG;
    }
    rtoss_device_guard on_device(ctx->device);   // the caller's current device comes back when the call returns
    cudaStream_t s = (cudaStream_t)cuda_stream;
    cudaError_t e = cudaSuccess;
    const unsigned cap = (unsigned)ctx->sm_count * 8u;
    if (b->n_chunks) {
        const unsigned grid = b->n_chunks < cap ? b->n_chunks : cap;
        e = rtoss_dev::launch_pdl(batch_select_pack_kernel, grid, kChunk, 0, s, (const BatchLayer*)b->layers_dev,
                                  (const uint32_t*)b->chunk_layer_dev, b->n_chunks);
    }
    if (e == cudaSuccess && b->n_tasks) {
        unsigned grid = (b->n_tasks + kOrderWarps - 1) / kOrderWarps;
        if (grid > cap) grid = cap;
        e = rtoss_dev::launch_pdl(batch_order_kernel, grid, kOrderWarps * 32, 0, s, (const BatchLayer*)b->layers_dev,
                                  (const uint32_t*)b->task_layer_dev, b->n_tasks);
    }
    if (e != cudaSuccess) {
        cudaGetLastError();
        snprintf(ctx->err, sizeof(ctx->err), "batch launch: %s", cudaGetErrorString(e));
        return RTOSS_ERR_CUDA;
    }
    return RTOSS_OK;
}

void rtoss_batch_destroy(rtoss_batch* b) {
    if (!b) return;
    int prev = 0;
    cudaGetDevice(&prev);
    cudaSetDevice(b->device);
    if (b->layers_dev) cudaFree(b->layers_dev);
    if (b->chunk_layer_dev) cudaFree(b->chunk_layer_dev);
    if (b->task_layer_dev) cudaFree(b->task_layer_dev);
    cudaSetDevice(prev);
    delete b;
}

}  // extern "C"
