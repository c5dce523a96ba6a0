// Pattern selection (Algorithm 2 / Algorithm 3 of arXiv 2303.02191) and the
// packing kernels.  All three are bandwidth-bound streaming passes over the
// weights: 9 values read per kernel, one byte (pid) or k values written.
#include <atomic>
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>

#include <cstring>

#include "conv_common.cuh"
#include "rtoss_internal.h"
#include "select_core.cuh"

namespace {

constexpr int kSelThreads = 256;  // kernels per block iteration

template <typename T> __device__ __forceinline__ float widen(T v);
template <> __device__ __forceinline__ float widen<float>(float v) { return v; }
template <> __device__ __forceinline__ float widen<__nv_bfloat16>(__nv_bfloat16 v) { return __bfloat162float(v); }
template <> __device__ __forceinline__ float widen<__half>(__half v) { return __half2float(v); }

template <typename T> __device__ __forceinline__ T narrow(float v);
template <> __device__ __forceinline__ float narrow<float>(float v) { return v; }
template <> __device__ __forceinline__ __nv_bfloat16 narrow<__nv_bfloat16>(float v) { return __float2bfloat16_rn(v); }
template <> __device__ __forceinline__ __half narrow<__half>(float v) { return __float2half_rn(v); }

// Copy the 9*count weights of `count` consecutive kernels starting at kernel
// `first` into shared memory, coalesced, 16 bytes per thread where the chunk is
// whole.  The base pointer is 16-byte aligned and a full chunk is a multiple
// of 16 bytes, so every full chunk starts on a 16-byte boundary.
template <typename T>
__device__ __forceinline__ void stage_kernels(const T* __restrict__ w, int64_t first, int count, T* smem) {
    const T* src = w + first * 9;
    constexpr int kVecElems = 16 / sizeof(T);
    if (count == kSelThreads) {
        const int nvec = kSelThreads * 9 / kVecElems;
        const uint4* s4 = reinterpret_cast<const uint4*>(src);
        uint4* d4 = reinterpret_cast<uint4*>(smem);
        for (int i = threadIdx.x; i < nvec; i += kSelThreads) d4[i] = __ldg(s4 + i);
    } else {
        for (int i = threadIdx.x; i < count * 9; i += kSelThreads) smem[i] = src[i];
    }
}

// One thread per kernel: squares in fp32, pattern sums in fp32 over ascending
// taps, first strictly larger sum wins.  __fmul_rn / __fadd_rn keep the
// compiler from contracting or reordering the arithmetic.
template <typename T>
__global__ void __launch_bounds__(kSelThreads) select_kernel(const T* __restrict__ w, int64_t n_kernels, MaskTable table,
                                                             int P, uint8_t* __restrict__ pid) {
    rtoss_dev::pdl_enter();
    __shared__ __align__(16) T sw[kSelThreads * 9];
    const int64_t n_chunks = (n_kernels + kSelThreads - 1) / kSelThreads;
    for (int64_t chunk = blockIdx.x; chunk < n_chunks; chunk += gridDim.x) {
        const int64_t first = chunk * kSelThreads;
        const int count = (int)min((int64_t)kSelThreads, n_kernels - first);
        __syncthreads();
        stage_kernels<T>(w, first, count, sw);
        __syncthreads();
        if ((int)threadIdx.x < count) {
            float v[9];
#pragma unroll
            for (int t = 0; t < 9; ++t) v[t] = widen<T>(sw[threadIdx.x * 9 + t]);
            const int best = rtoss_dev::select_best(v, table.m, P);
            pid[first + threadIdx.x] = (uint8_t)best;
        }
    }
}

// Gather the k kept values of each kernel (ascending tap order) and round them to the packed type; the handle's
// own copy of the pattern ids and, where it has them, the dense-expanded weights of the tensor path are written
// on the way.
template <typename T, typename V>
__global__ void __launch_bounds__(kSelThreads) pack_values_kernel(const T* __restrict__ w, int64_t n_kernels,
                                                                  MaskTable table, const uint8_t* pid, int k,
                                                                  V* __restrict__ val, uint8_t* pid_copy,
                                                                  V* __restrict__ wtc, int ksize, int Cin,
                                                                  rtoss_wtc_layout lay) {
    rtoss_dev::pdl_enter_handle_writer();
    __shared__ __align__(16) T sw[kSelThreads * 9];
    const int64_t n_chunks = (n_kernels + kSelThreads - 1) / kSelThreads;
    for (int64_t chunk = blockIdx.x; chunk < n_chunks; chunk += gridDim.x) {
        const int64_t first = chunk * kSelThreads;
        const int count = (int)min((int64_t)kSelThreads, n_kernels - first);
        __syncthreads();
        stage_kernels<T>(w, first, count, sw);
        __syncthreads();
        if ((int)threadIdx.x < count) {
            const int64_t i = first + threadIdx.x;
            const uint8_t id = pid[i];
            pid_copy[i] = id;
            float v[9];
#pragma unroll
            for (int t = 0; t < 9; ++t) v[t] = widen<T>(sw[threadIdx.x * 9 + t]);
            rtoss_dev::pack_one<V>(v, table.m[id], i, k, val, wtc, ksize, Cin, lay.rows, lay.rep_rows, lay.copies);
        }
    }
}

// Per input channel: stable counting sort of the filters by pattern id, one warp per channel.
constexpr int kOrderWarps = 4;
__global__ void __launch_bounds__(kOrderWarps * 32) pack_order_kernel(const uint8_t* __restrict__ pid, int Cout, int Cin,
                                                                      int P, uint32_t* __restrict__ perm,
                                                                      uint32_t* __restrict__ bucket_off,
                                                                      const uint16_t* __restrict__ masks,
                                                                      unsigned long long* __restrict__ issue, int cb_log2) {
    rtoss_dev::pdl_enter_handle_writer();
    __shared__ uint32_t fill_all[kOrderWarps][256];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int ci = blockIdx.x * kOrderWarps + warp;
    if (ci >= Cin) return;  // whole warp leaves together; no block-wide barrier below
    rtoss_dev::order_channel(pid, Cout, Cin, P, ci, perm, bucket_off, fill_all[warp], lane, masks, issue, cb_log2);
}

// Selection with one pattern per block of FB filters x CB input channels (a variant of Algorithm 2 in the spirit of
// Section IV.C's shared kernel masks): the pattern that retains the most energy of the whole block.  One CTA per
// block, one thread per filter of the block.  Arithmetic, fixed so that the ids are reproducible:
//   q = w*w rounded to fp32, widened to double;  r[co][t] = sum over the block's channels, ascending, in double;
//   E[t] = sum over the block's filters, ascending, of r[co][t];  S_p = sum over the taps of mask p, ascending, of E[t];
//   first strictly larger S_p wins (ties -> lowest id, a NaN sum never wins).
constexpr int kSharedMaxFB = 256;
template <typename T>
__global__ void __launch_bounds__(kSharedMaxFB) select_shared_kernel(const T* __restrict__ w, int Cout, int Cin, int FB, int CB,
                                                                      MaskTable table, int P, uint8_t* __restrict__ pid) {
    rtoss_dev::pdl_enter();
    __shared__ double r[kSharedMaxFB][9];
    __shared__ double E[9];
    __shared__ int s_best;
    const int nbc = (Cin + CB - 1) / CB, nbf = (Cout + FB - 1) / FB;
    for (int blk = blockIdx.x; blk < nbc * nbf; blk += gridDim.x) {
        const int co0 = (blk / nbc) * FB, ci0 = (blk % nbc) * CB;
        const int co1 = min(co0 + FB, Cout), ci1 = min(ci0 + CB, Cin);
        const int co = co0 + (int)threadIdx.x;
        if (co < co1) {
            double acc[9];
#pragma unroll
            for (int t = 0; t < 9; ++t) acc[t] = 0.0;
            const T* kw = w + ((size_t)co * Cin + ci0) * 9;
            for (int ci = ci0; ci < ci1; ++ci, kw += 9) {
#pragma unroll
                for (int t = 0; t < 9; ++t) {
                    const float v = widen<T>(kw[t]);
                    acc[t] = __dadd_rn(acc[t], (double)__fmul_rn(v, v));
                }
            }
#pragma unroll
            for (int t = 0; t < 9; ++t) r[threadIdx.x][t] = acc[t];
        }
        __syncthreads();
        if (threadIdx.x < 9) {
            double e = 0.0;
            for (int f = 0; f < co1 - co0; ++f) e = __dadd_rn(e, r[f][threadIdx.x]);
            E[threadIdx.x] = e;
        }
        __syncthreads();
        if (threadIdx.x == 0) {
            int best = 0;
            double best_s = 0.0;
            for (int p = 0; p < P; ++p) {
                const unsigned m = table.m[p];
                double sv = 0.0;
                for (int t = 0; t < 9; ++t)
                    if (m & (1u << t)) sv = __dadd_rn(sv, E[t]);
                if (p == 0) {
                    best_s = sv;
                } else if (sv > best_s || (best_s != best_s && sv == sv)) {
                    best = p;
                    best_s = sv;
                }
            }
            s_best = best;
        }
        __syncthreads();
        if (co < co1) {
            const uint8_t b = (uint8_t)s_best;
            for (int ci = ci0; ci < ci1; ++ci) pid[(size_t)co * Cin + ci] = b;
        }
        __syncthreads();
    }
}

// Dense masked weights from the packed form, one thread per dense element.
template <typename V>
__global__ void to_dense_kernel(const V* __restrict__ val, const uint8_t* __restrict__ pid,
                                const uint16_t* __restrict__ masks, int k, int64_t n_kernels, int64_t n_dense,
                                V* __restrict__ out) {
    rtoss_dev::pdl_enter();
    for (int64_t e = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; e < n_dense; e += (int64_t)gridDim.x * blockDim.x) {
        const int64_t g = e / 9;
        const int t = (int)(e - 9 * g);
        V v = narrow<V>(0.f);
        if (g < n_kernels) {
            const unsigned m = masks[pid[g]];
            if (m & (1u << t)) v = val[g * k + __popc(m & ((1u << t) - 1u))];
        }
        out[e] = v;
    }
}

int grid_for(int64_t n_chunks) {
    int64_t g = n_chunks < 1 ? 1 : n_chunks;
    const int64_t cap = 148 * 8;
    return (int)(g > cap ? cap : g);
}

}  // namespace

int rtoss_launch_select(const void* w, rtoss_dtype wdt, int64_t n_kernels, const MaskTable& t, int P, uint8_t* pid,
                        void* stream) {
    if (n_kernels <= 0) return 0;
    cudaStream_t s = (cudaStream_t)stream;
    const int grid = grid_for((n_kernels + kSelThreads - 1) / kSelThreads);
    switch (wdt) {
        case RTOSS_F32: rtoss_dev::launch_pdl(select_kernel<float>, grid, kSelThreads, 0, s, (const float*)w, n_kernels, t, P, pid); break;
        case RTOSS_BF16:
            rtoss_dev::launch_pdl(select_kernel<__nv_bfloat16>, grid, kSelThreads, 0, s, (const __nv_bfloat16*)w, n_kernels, t, P, pid);
            break;
        case RTOSS_F16: rtoss_dev::launch_pdl(select_kernel<__half>, grid, kSelThreads, 0, s, (const __half*)w, n_kernels, t, P, pid); break;
    }
    return (int)cudaGetLastError();
}

template <typename T>
static int launch_pack_values_t(const T* w, int64_t n, const MaskTable& t, const uint8_t* pid, int k, void* val,
                                rtoss_dtype vdt, uint8_t* pid_copy, void* wtc, int ksize, int Cin, rtoss_wtc_layout lay, cudaStream_t s) {
    const int grid = grid_for((n + kSelThreads - 1) / kSelThreads);
    switch (vdt) {
        case RTOSS_F32: rtoss_dev::launch_pdl(pack_values_kernel<T, float>, grid, kSelThreads, 0, s, w, n, t, pid, k, (float*)val, pid_copy, (float*)wtc, ksize, Cin, lay); break;
        case RTOSS_BF16:
            rtoss_dev::launch_pdl(pack_values_kernel<T, __nv_bfloat16>, grid, kSelThreads, 0, s, w, n, t, pid, k, (__nv_bfloat16*)val, pid_copy, (__nv_bfloat16*)wtc, ksize, Cin, lay);
            break;
        case RTOSS_F16: rtoss_dev::launch_pdl(pack_values_kernel<T, __half>, grid, kSelThreads, 0, s, w, n, t, pid, k, (__half*)val, pid_copy, (__half*)wtc, ksize, Cin, lay); break;
    }
    return (int)cudaGetLastError();
}

int rtoss_launch_pack_values(const void* w, rtoss_dtype wdt, int64_t n_kernels, const MaskTable& t, const uint8_t* pid,
                             int k, void* val, rtoss_dtype vdt, uint8_t* pid_copy, void* wtc, int ksize, int Cout, int Cin,
                             void* stream) {
    const rtoss_wtc_layout lay = rtoss_wtc_layout_of(Cout, ksize);
    if (n_kernels <= 0) return 0;
    cudaStream_t s = (cudaStream_t)stream;
    switch (wdt) {
        case RTOSS_F32: return launch_pack_values_t<float>((const float*)w, n_kernels, t, pid, k, val, vdt, pid_copy, wtc, ksize, Cin, lay, s);
        case RTOSS_BF16:
            return launch_pack_values_t<__nv_bfloat16>((const __nv_bfloat16*)w, n_kernels, t, pid, k, val, vdt, pid_copy, wtc, ksize, Cin, lay, s);
        case RTOSS_F16: return launch_pack_values_t<__half>((const __half*)w, n_kernels, t, pid, k, val, vdt, pid_copy, wtc, ksize, Cin, lay, s);
    }
    return (int)cudaErrorInvalidValue;
}

int rtoss_launch_pack_order(const uint8_t* pid, int Cout, int Cin, int P, uint32_t* perm, uint32_t* bucket_off,
                            const uint16_t* masks_dev, unsigned long long* issue, int cb_log2, void* stream) {
    const int grid = (Cin + kOrderWarps - 1) / kOrderWarps;
    rtoss_dev::launch_pdl(pack_order_kernel, grid, kOrderWarps * 32, 0, (cudaStream_t)stream, pid, Cout, Cin, P, perm, bucket_off,
                          masks_dev, issue, cb_log2);
    return (int)cudaGetLastError();
}

int rtoss_launch_select_shared(const void* w, rtoss_dtype wdt, int Cout, int Cin, int FB, int CB, const MaskTable& t, int P,
                               uint8_t* pid, void* stream) {
    cudaStream_t s = (cudaStream_t)stream;
    const int64_t blocks = (int64_t)((Cout + FB - 1) / FB) * ((Cin + CB - 1) / CB);
    const int grid = grid_for(blocks);
    const int threads = ((FB < Cout ? FB : Cout) + 31) / 32 * 32;
    cudaError_t e = cudaErrorInvalidValue;
    switch (wdt) {
        case RTOSS_F32: e = rtoss_dev::launch_pdl(select_shared_kernel<float>, grid, threads, 0, s, (const float*)w, Cout, Cin, FB, CB, t, P, pid); break;
        case RTOSS_BF16:
            e = rtoss_dev::launch_pdl(select_shared_kernel<__nv_bfloat16>, grid, threads, 0, s, (const __nv_bfloat16*)w, Cout, Cin, FB, CB, t, P, pid);
            break;
        case RTOSS_F16: e = rtoss_dev::launch_pdl(select_shared_kernel<__half>, grid, threads, 0, s, (const __half*)w, Cout, Cin, FB, CB, t, P, pid); break;
    }
    return (int)e;
}

int rtoss_launch_to_dense(const rtoss_packed* p, void* w_out, void* stream) {
    const int64_t n_dense = p->ksize == 3 ? p->n_kernels * 9 : (int64_t)p->Cout * p->Cin;
    if (n_dense <= 0) return 0;
    cudaStream_t s = (cudaStream_t)stream;
    const int threads = 256;
    const int grid = grid_for((n_dense + threads - 1) / threads);
    switch (p->dtype) {
        case RTOSS_F32:
            rtoss_dev::launch_pdl(to_dense_kernel<float>, grid, threads, 0, s, (const float*)p->val, p->pid, p->masks_dev, p->k, p->n_kernels,
                                                            n_dense, (float*)w_out);
            break;
        case RTOSS_BF16:
            rtoss_dev::launch_pdl(to_dense_kernel<__nv_bfloat16>, grid, threads, 0, s, (const __nv_bfloat16*)p->val, p->pid, p->masks_dev,
                                                                    p->k, p->n_kernels, n_dense, (__nv_bfloat16*)w_out);
            break;
        case RTOSS_F16:
            rtoss_dev::launch_pdl(to_dense_kernel<__half>, grid, threads, 0, s, (const __half*)p->val, p->pid, p->masks_dev, p->k,
                                                             p->n_kernels, n_dense, (__half*)w_out);
            break;
    }
    return (int)cudaGetLastError();
}

// ---------------------------------------------------------------------------------------------
// Pruning without any allocation.
//
// rtoss_select_patterns + rtoss_pack + rtoss_packed_to_dense produce the pruned dense weights
// W (.) mask, but rtoss_pack allocates the packed handle with cudaMalloc.  Some callers cannot do
// that: a serving process that handed all device memory to its own arena at start-up (a later
// cudaMalloc simply fails), or a control loop that may not take cudaMalloc / cudaFree's implicit
// device-wide synchronisation in the middle of its frames.  For them the pattern ids, the only
// intermediate of that chain, live in the fixed array below instead of a per-call buffer.
//
// The array is part of the library image: every GPU whose context loads the library holds
// kStaticPidBytes of device memory for it until the process exits.  All calls on a device share it.

constexpr size_t kStaticPidBytes = (size_t)1 << 20;  // one pattern id per kernel: at most 2^20 kernels per call
static __device__ __align__(256) unsigned char g_static_pid[kStaticPidBytes];

namespace {

// Dense masked weights straight from the weights and the pattern ids: out[e] = w[e] if position e is
// kept by the pattern of its kernel (or run of nine), else +0.
// w and out may be the same array (pruning in place): a thread reads element e and writes element e, nothing else,
// so neither pointer is declared restrict.
template <typename T>
__global__ void mask_dense_kernel(const T* w, const uint8_t* __restrict__ pid, MaskTable table,
                                  int64_t n_kernels, int64_t n_dense, T* out) {
    rtoss_dev::pdl_enter();
    for (int64_t e = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; e < n_dense; e += (int64_t)gridDim.x * blockDim.x) {
        const int64_t g = e / 9;
        const int t = (int)(e - 9 * g);
        T v = narrow<T>(0.f);
        if (g < n_kernels && (table.m[pid[g]] & (1u << t))) v = w[e];
        out[e] = v;
    }
}

// Device address of g_static_pid on the current device.  In host code the symbol's name is only a
// handle for the runtime, never a pointer a kernel could use: the address has to be asked for, once
// per device, with that device current.
unsigned char* static_pid_address(cudaError_t* err) {
    static std::atomic<unsigned char*> cached[64];   // two host threads may ask at once: both store the same address
    int dev = -1;
    *err = cudaGetDevice(&dev);
    if (*err != cudaSuccess) return nullptr;
    if (dev < 0 || dev >= 64) {
        *err = cudaErrorInvalidDevice;
        return nullptr;
    }
    unsigned char* at = cached[dev].load(std::memory_order_acquire);
    if (!at) {
        void* p = nullptr;
        *err = cudaGetSymbolAddress(&p, g_static_pid);
        if (*err != cudaSuccess) return nullptr;
        at = static_cast<unsigned char*>(p);
        cached[dev].store(at, std::memory_order_release);
    }
    return at;
}

}  // namespace

extern "C" rtoss_status rtoss_prune_dense_static(const void* w_dev, rtoss_dtype w_dtype, int Cout, int Cin, int ksize,
                                                 const uint16_t* masks_host, int P, int k, void* w_pruned_dev,
                                                 void* cuda_stream) {
    if (!w_dev || !w_pruned_dev || !masks_host) return RTOSS_ERR_INVALID_ARG;
    if (w_dtype != RTOSS_F32 && w_dtype != RTOSS_BF16 && w_dtype != RTOSS_F16) return RTOSS_ERR_INVALID_ARG;
    if (Cout < 1 || Cin < 1 || (ksize != 1 && ksize != 3)) return RTOSS_ERR_INVALID_ARG;
    if (!rtoss_table_ok(masks_host, P, k)) return RTOSS_ERR_BAD_PATTERN_TABLE;
    if ((reinterpret_cast<uintptr_t>(w_dev) & 15) || (reinterpret_cast<uintptr_t>(w_pruned_dev) & 15))
        return RTOSS_ERR_ALIGNMENT;
    const int64_t total = (int64_t)Cout * Cin;
    const int64_t n_kernels = ksize == 3 ? total : total / 9;
    if (n_kernels > (int64_t)kStaticPidBytes) return RTOSS_ERR_UNSUPPORTED;  // more kernels than the fixed array holds
    {
        // in place (same array) is fine; two different arrays that overlap are not
        const size_t bytes = (size_t)(ksize == 3 ? total * 9 : total) * rtoss_dtype_size(w_dtype);
        const uintptr_t a = reinterpret_cast<uintptr_t>(w_dev), b = reinterpret_cast<uintptr_t>(w_pruned_dev);
        if (a != b && a < b + bytes && b < a + bytes) return RTOSS_ERR_INVALID_ARG;
    }
    cudaError_t ce;
    unsigned char* pid = static_pid_address(&ce);
    if (!pid) return RTOSS_ERR_CUDA;
    MaskTable table;
    memset(&table, 0, sizeof(table));
    memcpy(table.m, masks_host, sizeof(uint16_t) * (size_t)P);
    // every pattern id this call reads is written by this call first: nothing in the array has to start at zero
    int e = rtoss_launch_select(w_dev, w_dtype, n_kernels, table, P, pid, cuda_stream);
    if (e) return RTOSS_ERR_CUDA;
    const int64_t n_dense = ksize == 3 ? total * 9 : total;
    const int threads = 256;
    const int grid = grid_for((n_dense + threads - 1) / threads);
    cudaStream_t s = (cudaStream_t)cuda_stream;
    cudaError_t le = cudaSuccess;   // this launch's own result (not the thread's last error, which may be older)
    switch (w_dtype) {
        case RTOSS_F32:
            le = rtoss_dev::launch_pdl(mask_dense_kernel<float>, grid, threads, 0, s, (const float*)w_dev, pid, table, n_kernels, n_dense, (float*)w_pruned_dev);
            break;
        case RTOSS_BF16:
            le = rtoss_dev::launch_pdl(mask_dense_kernel<__nv_bfloat16>, grid, threads, 0, s, (const __nv_bfloat16*)w_dev, pid, table, n_kernels, n_dense,
                                       (__nv_bfloat16*)w_pruned_dev);
            break;
        case RTOSS_F16:
            le = rtoss_dev::launch_pdl(mask_dense_kernel<__half>, grid, threads, 0, s, (const __half*)w_dev, pid, table, n_kernels, n_dense,
                                       (__half*)w_pruned_dev);
            break;
    }
    return le == cudaSuccess ? RTOSS_OK : RTOSS_ERR_CUDA;
}

// ---------------------------------------------------------------------------------------------
// Pattern usage ranking (Section IV.B, criterion 2): how often each pattern of a candidate table is the
// best fit over a sample of kernels.  The sample (random kernels in [-1, 1]) is the caller's input; this
// is the selection of Algorithm 2 followed by a histogram of the winning ids.
namespace {

__global__ void __launch_bounds__(256) pid_histogram_kernel(const uint8_t* __restrict__ pid, int64_t n, int P,
                                                            unsigned long long* __restrict__ counts) {
    rtoss_dev::pdl_enter();
    __shared__ unsigned int local[256];
    local[threadIdx.x] = 0;
    __syncthreads();
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (int64_t)gridDim.x * blockDim.x)
        atomicAdd(&local[pid[i]], 1u);
    __syncthreads();
    if ((int)threadIdx.x < P && local[threadIdx.x]) atomicAdd(&counts[threadIdx.x], (unsigned long long)local[threadIdx.x]);
}

}  // namespace

int rtoss_launch_pid_histogram(const uint8_t* pid, int64_t n, int P, unsigned long long* counts, void* stream) {
    if (n <= 0) return 0;
    rtoss_dev::launch_pdl(pid_histogram_kernel, grid_for((n + 255) / 256), 256, 0, (cudaStream_t)stream, pid, n, P, counts);
    return (int)cudaGetLastError();
}
