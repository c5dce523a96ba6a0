// Pattern-sparse 3x3 convolution on the FP32 FMA pipes.
//
// y = act(bias + sum over ci and over the k kept taps of kernel (co,ci)), the
// inference cost model of Section II.B of arXiv 2303.02191 (work proportional
// to the non-zero weights).  Because every kernel (co,ci) picks its own
// pattern, the kept (ci,tap) positions differ from filter to filter: this is a
// gather of k taps per kernel, not a dense contraction, and it runs on the
// plain FMA pipes.
//
// Shape of the kernel
//   * A CTA owns a spatial tile of one image and a block of kWarps*CO_T output
//     channels.  All warps share the staged input tile; warp w owns CO_T
//     consecutive filters, so the weights and the pattern a warp works on are
//     warp-uniform (one broadcast shared-memory read, uniform branches).
//   * Inside a warp, lane (lx,ly) of an LX x LY arrangement (LX*LY <= 32, picked
//     per layer by the host to waste the fewest lanes and pixels) owns a patch
//     of PH x PW output pixels and keeps its (PH-1)S+3 x (PW-1)S+3 input window
//     of the current input channel in registers.  That window is reused by the
//     CO_T filters of the warp.
//   * Per (filter, channel): the 9 dense-expanded weights and the pattern mask
//     are read once; each tap whose mask bit is set runs PH*PW FMAs with static
//     register indices; cleared taps are skipped by a uniform branch.  Only
//     k*PH*PW FMAs are issued per kernel.
//   * Input channels are staged CI_CHUNK at a time: activations converted to
//     fp32 once per tile (zero outside the image = the padding), weights
//     expanded from the packed (pid, k values) form into 9 slots + mask.
#include "conv_common.cuh"

namespace {

using namespace rtoss_dev;

constexpr int kWarps = 8;
constexpr int kThreads = kWarps * 32;
constexpr int kCiChunk = 8;
constexpr int kWSlots = 12;  // 9 weights, mask, 2 pad: three float4 per kernel

struct Conv3Args {
    const void* x;
    void* y;
    const void* val;
    const uint8_t* pid;
    const uint16_t* masks;
    const float* bias;
    int val_dtype;
    int N, Cin, Cout, H, W, Ho, Wo, k, P;
    int LX, LY, tiles_x, tiles_y;
    int TH_in, TW_in, TWP, plane;  // staged tile: rows, cols, row pitch, channel pitch (floats)
    int layout, act;
    int y_c_off, y_c_stride;
};

template <int S, int PH, int PW, int R, int C>
__device__ __forceinline__ void fma_tap(float (&acc)[PH][PW], const float (&win)[(PH - 1) * S + 3][(PW - 1) * S + 3],
                                        float w) {
#pragma unroll
    for (int py = 0; py < PH; ++py)
#pragma unroll
        for (int px = 0; px < PW; ++px) acc[py][px] = fmaf(w, win[py * S + R][px * S + C], acc[py][px]);
}

template <typename T, int S, int PH, int PW, int CO_T>
__global__ void __launch_bounds__(kThreads, 1) conv3x3_alu_kernel(const Conv3Args a) {
    constexpr int WIN_H = (PH - 1) * S + 3;
    constexpr int WIN_W = (PW - 1) * S + 3;
    constexpr int CO_BLOCK = kWarps * CO_T;

    extern __shared__ __align__(16) unsigned char smem_raw[];
    float* sX = reinterpret_cast<float*>(smem_raw);                        // [kCiChunk][plane]
    float* sW = sX + kCiChunk * a.plane;                                   // [kCiChunk][CO_BLOCK][kWSlots]
    int* tabG = reinterpret_cast<int*>(sW + kCiChunk * CO_BLOCK * kWSlots);  // [TH_in*TWP]
    __shared__ uint16_t smask[256];

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    int tile = blockIdx.x;
    const int tx = tile % a.tiles_x;
    tile /= a.tiles_x;
    const int ty = tile % a.tiles_y;
    const int n = tile / a.tiles_y;
    const int co0 = blockIdx.y * CO_BLOCK;

    const bool lane_active = lane < a.LX * a.LY;
    const int ly = lane_active ? lane / a.LX : 0;
    const int lx = lane_active ? lane - ly * a.LX : 0;
    const int ox0 = tx * a.LX * PW, oy0 = ty * a.LY * PH;  // first output pixel of the tile
    const int ix0 = ox0 * S - 1, iy0 = oy0 * S - 1;        // input coordinate of staged element (0,0)

    const int tile_elems = a.TH_in * a.TWP;
    for (int e = tid; e < tile_elems; e += kThreads) {
        const int r = e / a.TWP, c = e - r * a.TWP;
        const int iy = iy0 + r, ix = ix0 + c;
        const bool ok = c < a.TW_in && iy >= 0 && iy < a.H && ix >= 0 && ix < a.W;
        tabG[e] = ok ? iy * a.W + ix : -1;
    }
    for (int p = tid; p < 256; p += kThreads) smask[p] = p < a.P ? a.masks[p] : 0;

    float acc[CO_T][PH][PW];
#pragma unroll
    for (int c = 0; c < CO_T; ++c)
#pragma unroll
        for (int py = 0; py < PH; ++py)
#pragma unroll
            for (int px = 0; px < PW; ++px) acc[c][py][px] = 0.f;

    const T* __restrict__ xg = reinterpret_cast<const T*>(a.x);
    const size_t HW = (size_t)a.H * a.W;

    for (int ci0 = 0; ci0 < a.Cin; ci0 += kCiChunk) {
        __syncthreads();  // previous chunk fully consumed (also orders tabG / smask on the first pass)
        // ---- stage activations: fp32, zero where the tap falls outside the image
        if (a.layout == RTOSS_NCHW) {
            for (int cl = 0; cl < kCiChunk; ++cl) {
                const int ci = ci0 + cl;
                const T* plane_ptr = xg + ((size_t)n * a.Cin + (ci < a.Cin ? ci : 0)) * HW;
                float* dst = sX + cl * a.plane;
                for (int e = tid; e < tile_elems; e += kThreads) {
                    const int g = tabG[e];
                    dst[e] = (g >= 0 && ci < a.Cin) ? to_f32<T>(plane_ptr[g]) : 0.f;
                }
            }
        } else {
            const T* img = xg + (size_t)n * HW * a.Cin;
            for (int i = tid; i < tile_elems * kCiChunk; i += kThreads) {
                const int cl = i & (kCiChunk - 1), e = i >> 3;
                const int ci = ci0 + cl;
                const int g = tabG[e];
                sX[cl * a.plane + e] = (g >= 0 && ci < a.Cin) ? to_f32<T>(img[(size_t)g * a.Cin + ci]) : 0.f;
            }
        }
        // ---- stage weights: expand (pid, k values) to 9 slots + mask
        for (int i = tid; i < CO_BLOCK * kCiChunk; i += kThreads) {
            const int cl = i % kCiChunk, col = i / kCiChunk;
            const int co = co0 + col, ci = ci0 + cl;
            float wv[9];
#pragma unroll
            for (int t = 0; t < 9; ++t) wv[t] = 0.f;
            unsigned m = 0;
            if (co < a.Cout && ci < a.Cin) {
                const size_t kid = (size_t)co * a.Cin + ci;
                m = smask[a.pid[kid]];
                size_t j = kid * a.k;
#pragma unroll
                for (int t = 0; t < 9; ++t)
                    if (m & (1u << t)) wv[t] = load_val(a.val, j++, a.val_dtype);
            }
            float4* dst = reinterpret_cast<float4*>(sW + ((size_t)cl * CO_BLOCK + col) * kWSlots);
            dst[0] = make_float4(wv[0], wv[1], wv[2], wv[3]);
            dst[1] = make_float4(wv[4], wv[5], wv[6], wv[7]);
            dst[2] = make_float4(wv[8], __uint_as_float(m), 0.f, 0.f);
        }
        __syncthreads();

        // ---- compute
#pragma unroll 1
        for (int cl = 0; cl < kCiChunk; ++cl) {
            float win[WIN_H][WIN_W];
            const float* xp = sX + cl * a.plane + (ly * PH * S) * a.TWP + lx * PW * S;
#pragma unroll
            for (int r = 0; r < WIN_H; ++r) {
                const float* row = xp + r * a.TWP;
#pragma unroll
                for (int c4 = 0; c4 + 4 <= WIN_W; c4 += 4) {
                    const float4 v = *reinterpret_cast<const float4*>(row + c4);
                    win[r][c4] = v.x; win[r][c4 + 1] = v.y; win[r][c4 + 2] = v.z; win[r][c4 + 3] = v.w;
                }
#pragma unroll
                for (int c = (WIN_W / 4) * 4; c < WIN_W; ++c) win[r][c] = row[c];
            }
            const float4* wp = reinterpret_cast<const float4*>(sW + ((size_t)cl * CO_BLOCK + warp * CO_T) * kWSlots);
#pragma unroll
            for (int c = 0; c < CO_T; ++c) {
                const float4 w0 = wp[c * 3], w1 = wp[c * 3 + 1], w2 = wp[c * 3 + 2];
                const unsigned m = __float_as_uint(w2.y);
                if (m & 0x001) fma_tap<S, PH, PW, 0, 0>(acc[c], win, w0.x);
                if (m & 0x002) fma_tap<S, PH, PW, 0, 1>(acc[c], win, w0.y);
                if (m & 0x004) fma_tap<S, PH, PW, 0, 2>(acc[c], win, w0.z);
                if (m & 0x008) fma_tap<S, PH, PW, 1, 0>(acc[c], win, w0.w);
                if (m & 0x010) fma_tap<S, PH, PW, 1, 1>(acc[c], win, w1.x);
                if (m & 0x020) fma_tap<S, PH, PW, 1, 2>(acc[c], win, w1.y);
                if (m & 0x040) fma_tap<S, PH, PW, 2, 0>(acc[c], win, w1.z);
                if (m & 0x080) fma_tap<S, PH, PW, 2, 1>(acc[c], win, w1.w);
                if (m & 0x100) fma_tap<S, PH, PW, 2, 2>(acc[c], win, w2.x);
            }
        }
    }

    // ---- epilogue: bias, activation, rounding, store
    if (!lane_active) return;
    T* __restrict__ yg = reinterpret_cast<T*>(a.y);
    const int Cs = a.y_c_stride;
    const int ox_first = ox0 + lx * PW;
#pragma unroll
    for (int c = 0; c < CO_T; ++c) {
        const int co = co0 + warp * CO_T + c;
        if (co >= a.Cout) continue;
        const float b = a.bias ? a.bias[co] : 0.f;
#pragma unroll
        for (int py = 0; py < PH; ++py) {
            const int oy = oy0 + ly * PH + py;
            if (oy >= a.Ho) continue;
            if (a.layout == RTOSS_NCHW) {
                T* row = yg + (((size_t)n * Cs + a.y_c_off + co) * a.Ho + oy) * a.Wo;
                const bool vec = ((size_t)a.Wo * sizeof(T)) % 16 == 0 && ox_first + PW <= a.Wo && (PW * sizeof(T)) % 16 == 0;
                if (vec) {
                    T tmp[PW];
#pragma unroll
                    for (int px = 0; px < PW; ++px) tmp[px] = from_f32<T>(activate(acc[c][py][px] + b, a.act));
                    const uint4* src = reinterpret_cast<const uint4*>(tmp);
                    uint4* dst = reinterpret_cast<uint4*>(row + ox_first);
#pragma unroll
                    for (int v = 0; v < (int)(PW * sizeof(T) / 16); ++v) dst[v] = src[v];
                } else {
#pragma unroll
                    for (int px = 0; px < PW; ++px)
                        if (ox_first + px < a.Wo) row[ox_first + px] = from_f32<T>(activate(acc[c][py][px] + b, a.act));
                }
            } else {
#pragma unroll
                for (int px = 0; px < PW; ++px)
                    if (ox_first + px < a.Wo)
                        yg[(((size_t)n * a.Ho + oy) * a.Wo + ox_first + px) * Cs + a.y_c_off + co] =
                            from_f32<T>(activate(acc[c][py][px] + b, a.act));
            }
        }
    }
}

struct Variant {
    int S, PH, PW, CO_T;
};

// Pick the lane arrangement that wastes the fewest lanes and pixels.
void choose_lanes(int Ho, int Wo, int PH, int PW, int* LX, int* LY) {
    double best = -1.0;
    for (int lx = 1; lx <= 16; ++lx)
        for (int ly = 1; ly * lx <= 32; ++ly) {
            const int tw = lx * PW, th = ly * PH;
            const double cover = (double)((Wo + tw - 1) / tw * tw) * ((Ho + th - 1) / th * th);
            double util = (double)Wo * Ho / cover * (lx * ly) / 32.0;
            util -= 1e-3 * (double)(tw + th) / (tw * th);  // tie-break: less halo per pixel
            if (util > best) {
                best = util;
                *LX = lx;
                *LY = ly;
            }
        }
}

template <typename T, int S, int PH, int PW, int CO_T>
int launch_variant(Conv3Args& a, cudaStream_t stream) {
    choose_lanes(a.Ho, a.Wo, PH, PW, &a.LX, &a.LY);
    a.tiles_x = (a.Wo + a.LX * PW - 1) / (a.LX * PW);
    a.tiles_y = (a.Ho + a.LY * PH - 1) / (a.LY * PH);
    a.TW_in = (a.LX * PW - 1) * S + 3;
    a.TH_in = (a.LY * PH - 1) * S + 3;
    a.TWP = (a.TW_in + 3) / 4 * 4;
    const int elems = a.TH_in * a.TWP;
    a.plane = (elems + 31) / 32 * 32 + 4;
    const size_t smem = sizeof(float) * ((size_t)kCiChunk * a.plane + (size_t)kCiChunk * kWarps * CO_T * kWSlots) +
                        sizeof(int) * (size_t)elems;
    auto kern = conv3x3_alu_kernel<T, S, PH, PW, CO_T>;
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return (int)e;
    dim3 grid((unsigned)((size_t)a.tiles_x * a.tiles_y * a.N), (unsigned)((a.Cout + kWarps * CO_T - 1) / (kWarps * CO_T)));
    kern<<<grid, kThreads, smem, stream>>>(a);
    return (int)cudaGetLastError();
}

template <typename T>
int launch_typed(Conv3Args& a, int stride, cudaStream_t stream) {
    if (stride == 1) return launch_variant<T, 1, 4, 8, 4>(a, stream);
    return launch_variant<T, 2, 2, 8, 4>(a, stream);
}

}  // namespace

int rtoss_launch_conv3x3(const rtoss_ctx* ctx, const rtoss_packed* p, const void* x, void* y, const rtoss_conv_desc* d,
                         void* stream) {
    (void)ctx;
    Conv3Args a;
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
    a.Ho = (d->H - 1) / d->stride + 1;
    a.Wo = (d->W - 1) / d->stride + 1;
    a.k = p->k;
    a.P = p->P;
    a.layout = (int)d->layout;
    a.act = (int)d->act;
    a.y_c_off = d->y_channel_offset;
    a.y_c_stride = d->y_channel_stride ? d->y_channel_stride : p->Cout;
    cudaStream_t s = (cudaStream_t)stream;
    switch (d->io_dtype) {
        case RTOSS_F32: return launch_typed<float>(a, d->stride, s);
        case RTOSS_BF16: return launch_typed<__nv_bfloat16>(a, d->stride, s);
        case RTOSS_F16: return launch_typed<__half>(a, d->stride, s);
    }
    return (int)cudaErrorInvalidValue;
}
