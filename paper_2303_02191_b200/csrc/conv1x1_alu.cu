// Pattern-sparse 1x1 convolution on the FP32 FMA pipes.
//
// The 1x1 weights of a layer, flattened filter-major, were cut into runs of
// nine and each run pruned to the k taps of its pattern (Section IV.D,
// Algorithm 3 of arXiv 2303.02191).  Row co of the [Cout][Cin] matrix therefore
// keeps about Cin*k/9 entries at irregular positions: a sparse-matrix x
// dense-matrix product.  A thread keeps 8 x 16 accumulators (8 filters, 16
// pixels); per input channel it loads its 16 activations and the 8 weights
// (pruned ones are zeros) and issues all 128 FMAs.  Skipping the pruned
// weights with a uniform branch per (filter, channel) was measured and lost: a
// branch every 16-32 FMAs costs more than the zeros it avoids.  This is the
// path for fp32 and for what the tensor path does not take.
#include <atomic>

#include "conv_common.cuh"

namespace {

using namespace rtoss_dev;

constexpr int kWarps = 8;
constexpr int kThreads = kWarps * 32;
constexpr int kCiChunk = 32;  // channels per staging round: long enough to amortise the two barriers and the load latency
constexpr int kCoT = 8;
constexpr int kCoBlock = kWarps * kCoT;  // 64
constexpr int kPxThread = 16;
constexpr int kPxTile = 32 * kPxThread;  // 512 output pixels per CTA
constexpr int kXPitch = kPxTile + 4;     // floats per staged channel row: +4 keeps 16-byte alignment and spreads
                                         // eight consecutive channels over distinct banks

struct Conv1Args {
    const void* x;
    void* y;
    const void* val;
    const uint8_t* pid;
    const uint16_t* masks;
    const float* bias;
    int val_dtype;
    int N, Cin, Cout, H, W, Ho, Wo, k, P, stride;
    long long G;  // full runs of nine
    int tiles;    // pixel tiles per image
    int layout, act;
    int y_c_off, y_c_stride;
};

template <typename T>
__global__ void __launch_bounds__(kThreads, 1) conv1x1_alu_kernel(const Conv1Args a) {
    rtoss_dev::pdl_enter();
    extern __shared__ __align__(16) unsigned char smem_dyn[];
    float (*sX)[kXPitch] = reinterpret_cast<float (*)[kXPitch]>(smem_dyn);                                              // [kCiChunk][kXPitch]
    float (*sW)[kCoBlock] = reinterpret_cast<float (*)[kCoBlock]>(smem_dyn + sizeof(float) * kCiChunk * kXPitch);  // [kCiChunk][kCoBlock]
    __shared__ int tabG[kPxTile];
    __shared__ uint16_t smask[256];

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int n = blockIdx.x / a.tiles;
    const int tile = blockIdx.x - n * a.tiles;
    const int co0 = blockIdx.y * kCoBlock;
    const int HoWo = a.Ho * a.Wo;
    const int pix0 = tile * kPxTile;
    const size_t HW = (size_t)a.H * a.W;

    for (int e = tid; e < kPxTile; e += kThreads) {
        const int op = pix0 + e;
        int g = -1;
        if (op < HoWo) {
            const int oy = op / a.Wo, ox = op - oy * a.Wo;
            g = oy * a.stride * a.W + ox * a.stride;
        }
        tabG[e] = g;
    }
    for (int p = tid; p < 256; p += kThreads) smask[p] = p < a.P ? a.masks[p] : 0;

    float acc[kCoT][kPxThread];
#pragma unroll
    for (int c = 0; c < kCoT; ++c)
#pragma unroll
        for (int i = 0; i < kPxThread; ++i) acc[c][i] = 0.f;

    const T* __restrict__ xg = reinterpret_cast<const T*>(a.x);
    // contiguous fast path: NCHW, stride 1, whole tile inside the image, 16-byte aligned rows of the tile
    constexpr int kVec = 16 / sizeof(T);
    const bool fast = a.layout == RTOSS_NCHW && a.stride == 1 && pix0 + kPxTile <= HoWo && (HW % kVec) == 0;

    for (int ci0 = 0; ci0 < a.Cin; ci0 += kCiChunk) {
        __syncthreads();
        if (fast) {
            for (int i = tid; i < kCiChunk * (kPxTile / kVec); i += kThreads) {
                const int cl = i / (kPxTile / kVec), v = i - cl * (kPxTile / kVec);
                const int ci = ci0 + cl;
                float* dst = &sX[cl][v * kVec];
                if (ci < a.Cin) {
                    const uint4 raw = __ldg(reinterpret_cast<const uint4*>(xg + ((size_t)n * a.Cin + ci) * HW + pix0) + v);
                    const T* rv = reinterpret_cast<const T*>(&raw);
#pragma unroll
                    for (int q = 0; q < kVec; ++q) dst[q] = to_f32<T>(rv[q]);
                } else {
#pragma unroll
                    for (int q = 0; q < kVec; ++q) dst[q] = 0.f;
                }
            }
        } else if (a.layout == RTOSS_NCHW) {
            for (int cl = 0; cl < kCiChunk; ++cl) {
                const int ci = ci0 + cl;
                const T* plane_ptr = xg + ((size_t)n * a.Cin + (ci < a.Cin ? ci : 0)) * HW;
                for (int e = tid; e < kPxTile; e += kThreads) {
                    const int g = tabG[e];
                    sX[cl][e] = (g >= 0 && ci < a.Cin) ? to_f32<T>(plane_ptr[g]) : 0.f;
                }
            }
        } else {
            // NHWC: a warp takes eight consecutive channels of four pixels per step (16-byte runs in memory,
            // 32 distinct banks in shared memory)
            const T* img = xg + (size_t)n * HW * a.Cin;
            for (int cg = 0; cg < kCiChunk; cg += 8) {
                for (int i = tid; i < kPxTile * 8; i += kThreads) {
                    const int cl = cg + (i & 7), e = i >> 3;
                    const int ci = ci0 + cl;
                    const int g = tabG[e];
                    sX[cl][e] = (g >= 0 && ci < a.Cin) ? to_f32<T>(img[(size_t)g * a.Cin + ci]) : 0.f;
                }
            }
        }
        // weights of this chunk, dense-expanded: position (co, ci) holds its value or 0
        for (int i = tid; i < kCoBlock * kCiChunk; i += kThreads) {
            const int cl = i & (kCiChunk - 1), col = i / kCiChunk;
            const int co = co0 + col, ci = ci0 + cl;
            float w = 0.f;
            if (co < a.Cout && ci < a.Cin) {
                const long long e = (long long)co * a.Cin + ci;
                const long long g = e / 9;
                const int t = (int)(e - 9 * g);
                if (g < a.G) {
                    const unsigned m = smask[a.pid[g]];
                    if (m & (1u << t)) w = load_val(a.val, (size_t)(g * a.k + __popc(m & ((1u << t) - 1u))), a.val_dtype);
                }
            }
            sW[cl][col] = w;
        }
        __syncthreads();

#pragma unroll 2
        for (int cl = 0; cl < kCiChunk; ++cl) {
            float xv[kPxThread];
#pragma unroll
            for (int j = 0; j < kPxThread / 4; ++j) {
                const float4 v = *reinterpret_cast<const float4*>(&sX[cl][j * 128 + lane * 4]);
                xv[4 * j] = v.x; xv[4 * j + 1] = v.y; xv[4 * j + 2] = v.z; xv[4 * j + 3] = v.w;
            }
            const float4 wa = *reinterpret_cast<const float4*>(&sW[cl][warp * kCoT]);
            const float4 wb = *reinterpret_cast<const float4*>(&sW[cl][warp * kCoT + 4]);
            const float wv[kCoT] = {wa.x, wa.y, wa.z, wa.w, wb.x, wb.y, wb.z, wb.w};
#pragma unroll
            for (int c = 0; c < kCoT; ++c)
#pragma unroll
                for (int i = 0; i < kPxThread; ++i) acc[c][i] = fmaf(wv[c], xv[i], acc[c][i]);
        }
    }

    T* __restrict__ yg = reinterpret_cast<T*>(a.y);
    const int Cs = a.y_c_stride;
#pragma unroll
    for (int c = 0; c < kCoT; ++c) {
        const int co = co0 + warp * kCoT + c;
        if (co >= a.Cout) continue;
        const float b = a.bias ? a.bias[co] : 0.f;
#pragma unroll
        for (int j = 0; j < kPxThread / 4; ++j) {
            const int op = pix0 + j * 128 + lane * 4;
            if (op >= HoWo) continue;
            if (a.layout == RTOSS_NCHW) {
                T* dst = yg + ((size_t)n * Cs + a.y_c_off + co) * HoWo + op;
                if ((HoWo & 3) == 0) {  // op is a multiple of 4 and so is every plane start: aligned 4-element store
                    __align__(16) T tmp[4];
#pragma unroll
                    for (int q = 0; q < 4; ++q) tmp[q] = from_f32<T>(activate(acc[c][4 * j + q] + b, a.act));
                    if (sizeof(T) == 4) *reinterpret_cast<uint4*>(dst) = *reinterpret_cast<const uint4*>(tmp);
                    else *reinterpret_cast<uint2*>(dst) = *reinterpret_cast<const uint2*>(tmp);
                } else {
#pragma unroll
                    for (int q = 0; q < 4; ++q)
                        if (op + q < HoWo) dst[q] = from_f32<T>(activate(acc[c][4 * j + q] + b, a.act));
                }
            } else {
#pragma unroll
                for (int q = 0; q < 4; ++q)
                    if (op + q < HoWo)
                        yg[((size_t)n * HoWo + op + q) * Cs + a.y_c_off + co] =
                            from_f32<T>(activate(acc[c][4 * j + q] + b, a.act));
            }
        }
    }
}

}  // namespace

int rtoss_launch_conv1x1(const rtoss_ctx* ctx, const rtoss_packed* p, const void* x, void* y, const rtoss_conv_desc* d,
                         void* stream) {
    (void)ctx;
    Conv1Args a;
    a.x = x;
    a.y = y;
    a.val = p->val;
    a.pid = p->pid;
    a.masks = p->masks_dev;
    a.bias = d->bias_dev;
    a.val_dtype = (int)p->dtype;
    a.N = d->N;
    a.Cin = p->Cin;
    a.Cout = p->Cout;
    a.H = d->H;
    a.W = d->W;
    a.stride = d->stride;
    a.Ho = (d->H - 1) / d->stride + 1;
    a.Wo = (d->W - 1) / d->stride + 1;
    a.k = p->k;
    a.P = p->P;
    a.G = p->n_kernels;
    a.tiles = (a.Ho * a.Wo + kPxTile - 1) / kPxTile;
    a.layout = (int)d->layout;
    a.act = (int)d->act;
    a.y_c_off = d->y_channel_offset;
    a.y_c_stride = d->y_channel_stride ? d->y_channel_stride : p->Cout;
    dim3 grid((unsigned)((size_t)a.tiles * a.N), (unsigned)((a.Cout + kCoBlock - 1) / kCoBlock));
    cudaStream_t s = (cudaStream_t)stream;
    const int smem = (int)sizeof(float) * kCiChunk * (kXPitch + kCoBlock);
    // the attribute belongs to the (function, device) pair: one flag per device
    static std::atomic<bool> attr_set[64];
    const int dev_slot = ctx->device >= 0 && ctx->device < 64 ? ctx->device : -1;
    if (dev_slot < 0 || !attr_set[dev_slot].load(std::memory_order_acquire)) {
        cudaError_t e = cudaFuncSetAttribute(conv1x1_alu_kernel<float>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
        if (e == cudaSuccess) e = cudaFuncSetAttribute(conv1x1_alu_kernel<__nv_bfloat16>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
        if (e == cudaSuccess) e = cudaFuncSetAttribute(conv1x1_alu_kernel<__half>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
        if (e != cudaSuccess) return (int)e;
        if (dev_slot >= 0) attr_set[dev_slot].store(true, std::memory_order_release);
    }
    switch (d->io_dtype) {
        case RTOSS_F32: rtoss_dev::launch_pdl(conv1x1_alu_kernel<float>, grid, kThreads, smem, s, a); break;
        case RTOSS_BF16: rtoss_dev::launch_pdl(conv1x1_alu_kernel<__nv_bfloat16>, grid, kThreads, smem, s, a); break;
        case RTOSS_F16: rtoss_dev::launch_pdl(conv1x1_alu_kernel<__half>, grid, kThreads, smem, s, a); break;
    }
    return (int)cudaGetLastError();
}
