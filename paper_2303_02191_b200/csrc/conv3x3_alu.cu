// Pattern-sparse 3x3 convolution on the FP32 FMA pipes.
//
// y = act(bias + sum over ci and over the k kept taps of kernel (co,ci)), the
// inference cost model of Section II.B of arXiv 2303.02191 (work proportional
// to the non-zero weights).  Because every kernel (co,ci) picks its own
// pattern, the kept (ci,tap) positions differ from filter to filter: this is a
// gather of k taps per kernel, not a dense contraction.  This path runs it on
// the plain FMA pipes (any dtype, layout and stride; the only path for fp32).
//
// Shape of the kernel
//   * A CTA owns a spatial tile of one image and a block of WARPS*CO_T output
//     channels.  All warps share the staged input tile; warp w owns CO_T
//     consecutive filters, so the weights a warp works on are warp-uniform
//     (one broadcast shared-memory read; no branch depends on the pattern).
//   * Inside a warp, lane (lx,ly) of an LX x LY arrangement (LX*LY <= 32, picked
//     per layer by the host to waste the fewest lanes and pixels) owns a patch
//     of PH x PW output pixels and keeps its (PH-1)S+3 x (PW-1)S+3 input window
//     of the current input channel in registers.  That window is reused by the
//     CO_T filters of the warp.
//   * Per (filter, channel): the 9 dense-expanded weights (pruned taps = 0) are
//     read once and all nine taps run PH*PW FMAs with static register indices.
//     The sparsity is not skipped here (see the note in the compute loop); it
//     pays through the packed weights' smaller HBM footprint only.
//   * Input channels are processed kCiChunk at a time through a two-stage
//     pipeline: while chunk i is being computed, the raw bytes of chunk i+1
//     (activations in their storage type, packed values and pattern ids) arrive
//     in shared memory through cp.async.  Before computing a chunk its raw bytes
//     are converted once: activations to fp32 (zero outside the image = the
//     padding), weights from (pid, k values) to 9 slots + mask.
//   * cp.async needs aligned rows.  NCHW: image rows must start on a multiple of
//     4, 8 or 16 bytes (the widest that divides W*elem is used); NHWC: Cin a
//     multiple of 8.  Weights: Cin a multiple of 8.  Anything else takes a plain
//     load-convert-store path inside the same kernel.
#include <cstring>

#include "conv_common.cuh"

namespace {

using namespace rtoss_dev;

constexpr int kCiChunk = 8;
constexpr int kWSlots = 12;  // 9 weights, mask, 2 pad: three float4 per kernel

enum XMode { X_SYNC = 0, X_NCHW_VEC = 1, X_NHWC_VEC = 2 };

struct Conv3Args {
    const void* x;
    void* y;
    const void* val;
    const uint8_t* pid;
    const uint16_t* masks;
    const float* bias;
    int val_dtype, val_esize;
    int N, Cin, Cout, H, W, Ho, Wo, k, P;
    int LX, LY, tiles_x, tiles_y;
    int TH_in, TW_in, TWP, plane;  // staged fp32 tile: rows, cols, row pitch, channel pitch (floats)
    int xmode;                     // XMode
    int vb;                        // bytes per cp.async of activations (4, 8, 16)
    int EV;                        // raw vectors per channel plane (NCHW) or pixels per tile (NHWC)
    int w_async;                   // packed weights arrive through cp.async
    int layout, act;
    int y_c_off, y_c_stride;
    // byte offsets of the shared-memory regions
    int off_sW, off_rawX, rawX_bytes, off_rawV, rawV_bytes, off_rawP, off_tab;
};

__device__ __forceinline__ void cp_async(void* smem_dst, const void* gsrc, int bytes) {
    const unsigned s = (unsigned)__cvta_generic_to_shared(smem_dst);
    if (bytes == 16) asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(s), "l"(gsrc) : "memory");
    else if (bytes == 8) asm volatile("cp.async.ca.shared.global [%0], [%1], 8;" ::"r"(s), "l"(gsrc) : "memory");
    else asm volatile("cp.async.ca.shared.global [%0], [%1], 4;" ::"r"(s), "l"(gsrc) : "memory");
}
__device__ __forceinline__ void cp_async_wait_all() { asm volatile("cp.async.wait_all;" ::: "memory"); }

template <int S, int PH, int PW, int R, int C>
__device__ __forceinline__ void fma_tap(float (&acc)[PH][PW], const float (&win)[(PH - 1) * S + 3][(PW - 1) * S + 3],
                                        float w) {
#pragma unroll
    for (int py = 0; py < PH; ++py)
#pragma unroll
        for (int px = 0; px < PW; ++px) acc[py][px] = fmaf(w, win[py * S + R][px * S + C], acc[py][px]);
}

template <int VB>
__device__ __forceinline__ void cp_async_fixed(void* smem_dst, const void* gsrc) {
    const unsigned s = (unsigned)__cvta_generic_to_shared(smem_dst);
    if (VB == 16) asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(s), "l"(gsrc) : "memory");
    else if (VB == 8) asm volatile("cp.async.ca.shared.global [%0], [%1], 8;" ::"r"(s), "l"(gsrc) : "memory");
    else asm volatile("cp.async.ca.shared.global [%0], [%1], 4;" ::"r"(s), "l"(gsrc) : "memory");
}

// NCHW activations of one chunk: a thread owns raw vector e of EVERY channel of the chunk, so the table
// entry is read once and the eight copies are independent of one another.
template <typename T, int VB, int NTHREADS>
__device__ __forceinline__ void issue_nchw(const T* chunk_base, size_t HW, int n_ch, const int* tab_g, int EV,
                                           unsigned char* dst, int tid) {
    for (int e = tid; e < EV; e += NTHREADS) {
        const int g = tab_g[e];
        if (g < 0) continue;
        const T* src = chunk_base + g;
        unsigned char* d = dst + (size_t)e * VB;
#pragma unroll
        for (int cl = 0; cl < kCiChunk; ++cl)
            if (cl < n_ch) cp_async_fixed<VB>(d + (size_t)cl * EV * VB, src + (size_t)cl * HW);
    }
}

// Conversion of the raw vectors into the fp32 tile, same ownership: table entries and the destination
// bounds are worked out once per vector, then applied to the eight channels.
template <typename T, int VB, int NTHREADS>
__device__ __forceinline__ void convert_nchw(const unsigned char* src, int n_ch, const int* tab_g, const int* tab_s, int EV,
                                             float* sX, int plane, int TWP, int tid) {
    constexpr int VEQ = VB / (int)sizeof(T);
    for (int e = tid; e < EV; e += NTHREADS) {
        const bool inside = tab_g[e] >= 0;
        const int s = tab_s[e];
        const int r = s >> 16, c0 = (s & 0xFFFF) - 16;  // destination row, column of element 0 (>= -(VEQ-1))
        float* drow = sX + r * TWP + c0;
#pragma unroll
        for (int cl = 0; cl < kCiChunk; ++cl) {
            const bool ok = inside && cl < n_ch;
            __align__(16) T v[VEQ];
            if (VB == 16) *reinterpret_cast<uint4*>(v) = *reinterpret_cast<const uint4*>(src + ((size_t)cl * EV + e) * VB);
            else if (VB == 8) *reinterpret_cast<uint2*>(v) = *reinterpret_cast<const uint2*>(src + ((size_t)cl * EV + e) * VB);
            else *reinterpret_cast<unsigned*>(v) = *reinterpret_cast<const unsigned*>(src + ((size_t)cl * EV + e) * VB);
#pragma unroll
            for (int q = 0; q < VEQ; ++q) {
                const int c = c0 + q;
                if (c >= 0 && c < TWP) drow[cl * plane + q] = ok ? to_f32<T>(v[q]) : 0.f;
            }
        }
    }
}

template <typename T, int S, int PH, int PW, int CO_T, int WARPS, int MINB>
__global__ void __launch_bounds__(WARPS * 32, MINB) conv3x3_alu_kernel(const Conv3Args a) {
    rtoss_dev::pdl_enter();
    constexpr int kThreads = WARPS * 32;
    constexpr int WIN_H = (PH - 1) * S + 3;
    constexpr int WIN_W = (PW - 1) * S + 3;
    constexpr int CO_BLOCK = WARPS * CO_T;

    constexpr int VE16 = 16 / (int)sizeof(T);
    static_assert(kCiChunk == 8, "index arithmetic below assumes chunks of 8 channels");

    extern __shared__ __align__(16) unsigned char smem[];
    float* sX = reinterpret_cast<float*>(smem);             // [kCiChunk][plane]
    float* sW = reinterpret_cast<float*>(smem + a.off_sW);   // [kCiChunk][CO_BLOCK][kWSlots]
    unsigned char* rawX = smem + a.off_rawX;                 // [2][rawX_bytes]
    unsigned char* rawV = smem + a.off_rawV;                 // [2][CO_BLOCK][8*k*val_esize]
    unsigned char* rawP = smem + a.off_rawP;                 // [2][CO_BLOCK][8]
    int* tab_g = reinterpret_cast<int*>(smem + a.off_tab);   // global element offset per table entry, -1 = outside
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

    // ---- tables, built once per CTA
    // X_SYNC / X_NHWC_VEC: one entry per staged element (r, c) of a channel plane, pitch TWP / TW_in;
    //             tab_s = its offset in the fp32 plane.
    // X_NCHW_VEC: one entry per raw vector (r, j); tab_g = offset of its first element in the channel
    //             plane, tab_s = its row packed with the (biased) destination column of its first element,
    //             which may lie left of the tile.
    const int veq = a.vb / (int)sizeof(T);  // elements per activation vector (NCHW vector mode)
    const int n_tab = a.xmode == X_SYNC ? a.TH_in * a.TWP : a.EV;
    int* tab_s = tab_g + n_tab;
    if (a.xmode == X_NCHW_VEC) {
        const int nv = a.EV / a.TH_in;
        for (int e = tid; e < n_tab; e += kThreads) {
            const int r = e / nv, j = e - r * nv;
            const int iy = iy0 + r, ix = ox0 * S - veq + j * veq;
            tab_g[e] = (iy >= 0 && iy < a.H && ix >= 0 && ix < a.W) ? iy * a.W + ix : -1;
            tab_s[e] = (r << 16) | (j * veq - (veq - 1) + 16);
        }
    } else {
        const int pitch = a.xmode == X_SYNC ? a.TWP : a.TW_in;
        for (int e = tid; e < n_tab; e += kThreads) {
            const int r = e / pitch, c = e - r * pitch;
            const int iy = iy0 + r, ix = ix0 + c;
            const bool ok = c < a.TW_in && iy >= 0 && iy < a.H && ix >= 0 && ix < a.W;
            tab_g[e] = ok ? iy * a.W + ix : -1;
            tab_s[e] = r * a.TWP + c;
        }
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
    const int vrow_bytes = 8 * a.k * a.val_esize;  // packed values of 8 consecutive channels of one filter
    __syncthreads();                                // tables visible before the first issue

    // ---- asynchronous part of staging chunk ci0 into raw buffer `buf`
    auto issue = [&](int ci0, int buf) {
        if (a.xmode == X_NCHW_VEC) {
            const int n_ch = a.Cin - ci0 < kCiChunk ? a.Cin - ci0 : kCiChunk;
            const T* chunk_base = xg + ((size_t)n * a.Cin + ci0) * HW;
            unsigned char* dst = rawX + (size_t)buf * a.rawX_bytes;
            if (a.vb == 16) issue_nchw<T, 16, kThreads>(chunk_base, HW, n_ch, tab_g, a.EV, dst, tid);
            else if (a.vb == 8) issue_nchw<T, 8, kThreads>(chunk_base, HW, n_ch, tab_g, a.EV, dst, tid);
            else issue_nchw<T, 4, kThreads>(chunk_base, HW, n_ch, tab_g, a.EV, dst, tid);
        } else if (a.xmode == X_NHWC_VEC) {
            constexpr int VPP = 8 / VE16;  // 16-byte vectors per pixel for 8 channels
            const T* img = xg + (size_t)n * HW * a.Cin + ci0;
            unsigned char* dst = rawX + (size_t)buf * a.rawX_bytes;
            for (int i = tid; i < a.EV * VPP; i += kThreads) {
                const int e = i / VPP, h = i - e * VPP;
                const int g = tab_g[e];
                if (g >= 0) cp_async(dst + (size_t)i * 16, img + (size_t)g * a.Cin + h * VE16, 16);
            }
        }
        if (a.w_async) {
            const int nvw = vrow_bytes / 16;
            unsigned char* dv = rawV + (size_t)buf * a.rawV_bytes;
            for (int i = tid; i < CO_BLOCK * nvw; i += kThreads) {
                const int col = i / nvw, j = i - col * nvw;
                const int co = co0 + col;
                if (co < a.Cout)
                    cp_async(dv + (size_t)col * vrow_bytes + j * 16,
                             reinterpret_cast<const unsigned char*>(a.val) +
                                 ((size_t)co * a.Cin + ci0) * a.k * a.val_esize + j * 16, 16);
            }
            if (tid < CO_BLOCK && co0 + tid < a.Cout)
                cp_async(rawP + (size_t)buf * CO_BLOCK * 8 + tid * 8, a.pid + (size_t)(co0 + tid) * a.Cin + ci0, 8);
        }
        asm volatile("cp.async.commit_group;" ::: "memory");
    };

    // ---- conversion of chunk ci0 (raw buffer `buf`, or straight from global memory) into sX / sW
    auto convert = [&](int ci0, int buf) {
        if (a.xmode == X_NCHW_VEC) {
            const int n_ch = a.Cin - ci0 < kCiChunk ? a.Cin - ci0 : kCiChunk;
            const unsigned char* src = rawX + (size_t)buf * a.rawX_bytes;
            if (a.vb == 16) convert_nchw<T, 16, kThreads>(src, n_ch, tab_g, tab_s, a.EV, sX, a.plane, a.TWP, tid);
            else if (a.vb == 8) {
                if (sizeof(T) <= 4) convert_nchw<T, 8, kThreads>(src, n_ch, tab_g, tab_s, a.EV, sX, a.plane, a.TWP, tid);
            } else {
                if (sizeof(T) <= 4) convert_nchw<T, 4, kThreads>(src, n_ch, tab_g, tab_s, a.EV, sX, a.plane, a.TWP, tid);
            }
        } else if (a.xmode == X_NHWC_VEC) {
            const unsigned char* src = rawX + (size_t)buf * a.rawX_bytes;
            for (int e = tid; e < a.EV; e += kThreads) {
                const bool ok = tab_g[e] >= 0;
                const int s = tab_s[e];
                const T* rv = reinterpret_cast<const T*>(src + (size_t)e * (8 * sizeof(T)));
#pragma unroll
                for (int cl = 0; cl < 8; ++cl) sX[cl * a.plane + s] = ok ? to_f32<T>(rv[cl]) : 0.f;
            }
        } else if (a.layout == RTOSS_NCHW) {
            const int tile_elems = a.TH_in * a.TWP;
            for (int cl = 0; cl < kCiChunk; ++cl) {
                const int ci = ci0 + cl;
                const T* plane_ptr = xg + ((size_t)n * a.Cin + (ci < a.Cin ? ci : 0)) * HW;
                float* dst = sX + cl * a.plane;
                for (int e = tid; e < tile_elems; e += kThreads) {
                    const int g = tab_g[e];
                    dst[e] = (g >= 0 && ci < a.Cin) ? to_f32<T>(plane_ptr[g]) : 0.f;
                }
            }
        } else {
            const int tile_elems = a.TH_in * a.TWP;
            const T* img = xg + (size_t)n * HW * a.Cin;
            for (int i = tid; i < tile_elems * kCiChunk; i += kThreads) {
                const int cl = i & (kCiChunk - 1), e = i >> 3;
                const int ci = ci0 + cl;
                const int g = tab_g[e];
                sX[cl * a.plane + e] = (g >= 0 && ci < a.Cin) ? to_f32<T>(img[(size_t)g * a.Cin + ci]) : 0.f;
            }
        }
        // weights: expand (pid, k values) of each (filter, channel) of the chunk to 9 slots + mask
        for (int i = tid; i < CO_BLOCK * kCiChunk; i += kThreads) {
            const int cl = i % kCiChunk, col = i / kCiChunk;
            const int co = co0 + col, ci = ci0 + cl;
            float wv[9];
#pragma unroll
            for (int t = 0; t < 9; ++t) wv[t] = 0.f;
            unsigned m = 0;
            if (co < a.Cout && ci < a.Cin) {
                if (a.w_async) {
                    m = smask[rawP[(size_t)buf * CO_BLOCK * 8 + col * 8 + cl]];
                    const void* vals = rawV + (size_t)buf * a.rawV_bytes + (size_t)col * vrow_bytes;
                    int j = cl * a.k;
#pragma unroll
                    for (int t = 0; t < 9; ++t)
                        if (m & (1u << t)) wv[t] = load_val(vals, j++, a.val_dtype);
                } else {
                    const size_t kid = (size_t)co * a.Cin + ci;
                    m = smask[a.pid[kid]];
                    size_t j = kid * a.k;
#pragma unroll
                    for (int t = 0; t < 9; ++t)
                        if (m & (1u << t)) wv[t] = load_val(a.val, j++, a.val_dtype);
                }
            }
            float4* dst = reinterpret_cast<float4*>(sW + ((size_t)cl * CO_BLOCK + col) * kWSlots);
            dst[0] = make_float4(wv[0], wv[1], wv[2], wv[3]);
            dst[1] = make_float4(wv[4], wv[5], wv[6], wv[7]);
            dst[2] = make_float4(wv[8], __uint_as_float(m), 0.f, 0.f);
        }
    };

    const int n_chunks = (a.Cin + kCiChunk - 1) / kCiChunk;
    issue(0, 0);
    for (int ch = 0; ch < n_chunks; ++ch) {
        cp_async_wait_all();
        __syncthreads();  // raw bytes of this chunk visible to all; everyone is done computing the previous chunk
        if (ch + 1 < n_chunks) issue((ch + 1) * kCiChunk, (ch + 1) & 1);
        convert(ch * kCiChunk, ch & 1);
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
            // the weights of filter c+1 are fetched before the FMAs of filter c, so the shared-memory
            // latency is covered by arithmetic instead of being exposed at every filter
            float4 n0 = wp[0], n1 = wp[1], n2 = wp[2];
#pragma unroll
            for (int c = 0; c < CO_T; ++c) {
                const float4 w0 = n0, w1 = n1, w2 = n2;
                if (c + 1 < CO_T) {
                    n0 = wp[(c + 1) * 3];
                    n1 = wp[(c + 1) * 3 + 1];
                    n2 = wp[(c + 1) * 3 + 2];
                }
                // All nine taps, no branch: the pruned taps of a kernel are zeros in its expanded weights.
                // Skipping them was measured and lost: with one pattern per (filter, channel) a skip is a
                // branch every few dozen FMAs, and the dispatch instructions plus the instruction-fetch
                // stalls after taken branches cost as much as the multiplications they avoid.
                fma_tap<S, PH, PW, 0, 0>(acc[c], win, w0.x);
                fma_tap<S, PH, PW, 0, 1>(acc[c], win, w0.y);
                fma_tap<S, PH, PW, 0, 2>(acc[c], win, w0.z);
                fma_tap<S, PH, PW, 1, 0>(acc[c], win, w0.w);
                fma_tap<S, PH, PW, 1, 1>(acc[c], win, w1.x);
                fma_tap<S, PH, PW, 1, 2>(acc[c], win, w1.y);
                fma_tap<S, PH, PW, 2, 0>(acc[c], win, w1.z);
                fma_tap<S, PH, PW, 2, 1>(acc[c], win, w1.w);
                fma_tap<S, PH, PW, 2, 2>(acc[c], win, w2.x);
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
                    __align__(16) T tmp[PW];
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

// ---------------------------------------------------------------------------------------------
// Layers with very few input channels (the 3-channel stem of a detector).  A thread computes kStemPx
// neighbouring output pixels of one row for 32 filters: its input window (3 rows x ((kStemPx-1)*S+3)
// columns x CIN) sits in registers, the dense-expanded weights (pruned taps are zeros: with 9*CIN <= 36
// multiply-adds per output the zeros cost less than skipping them) are read from shared memory once per
// filter as 16-byte loads and used for all kStemPx pixels.  The layer's bound is its traffic, so loads and
// stores must be whole segments:
//   * the detector stem proper (three 16-bit channels, NHWC, stride 2, rows of a multiple of 8 pixels): a
//     thread's window of 9 pixels x 3 channels is 54 contiguous bytes that start 6 bytes before a 16-byte
//     boundary, so it comes in as four aligned 16-byte loads per row and every value sits at a position
//     known at compile time (81 separate 2-byte loads a thread, each lane in its own sector, were what
//     bounded the kernel before);
//   * with 16-bit NHWC outputs a block's 512 pixels x 32 filters are gathered in shared memory and written
//     out with consecutive lanes on consecutive 16 bytes.
// A block walks the pixel groups in steps of the grid, so the weight table is built once per block.
constexpr int kStemCo = 32;
constexpr int kStemPx = 4;
constexpr int kStemThreads = 128;
constexpr int kStemNf = 4;   // filters per trip of the filter loop

// SiLU of a 16-bit output through tanh.approx (relative error about 2^-11, below half an ulp of bf16);
// fp32 outputs keep the exponential form (the tolerance there is 1e-4).
template <typename T>
__device__ __forceinline__ float stem_act(float v, int act) {
    if (sizeof(T) == 2 && act == RTOSS_ACT_SILU) {
        const float h = 0.5f * v;
        float th;
        asm("tanh.approx.f32 %0, %1;" : "=f"(th) : "f"(h));
        return fmaf(h, th, h);
    }
    return activate(v, act);
}

template <typename T, int CIN, int S>
__global__ void __launch_bounds__(kStemThreads) conv3x3_small_cin_kernel(const Conv3Args a) {
    rtoss_dev::pdl_enter();
    constexpr int KW = (CIN * 9 + 1 + 3) / 4 * 4;          // a filter's row: CIN*9 weights, the bias, padding to 16 bytes
    constexpr int WIN = (kStemPx - 1) * S + 3;              // input columns a thread needs
    constexpr int kStageRow = kStemPx * 4 + 1;              // 16-byte pieces a thread stages (+1: lanes on different banks)
    __shared__ __align__(16) float sWd[kStemCo][KW];         // [filter][ci*9 + tap], then the bias
    __shared__ uint16_t smask[256];
    __shared__ uint4 sOut[sizeof(T) == 2 ? kStemThreads * kStageRow : 1];
    const int co0 = blockIdx.y * kStemCo;
    for (int p = threadIdx.x; p < 256; p += blockDim.x) smask[p] = p < a.P ? a.masks[p] : 0;
    __syncthreads();
    for (int i = threadIdx.x; i < kStemCo * CIN; i += blockDim.x) {
        const int col = i / CIN, ci = i - col * CIN, co = co0 + col;
        float wv[9];
#pragma unroll
        for (int t = 0; t < 9; ++t) wv[t] = 0.f;
        if (co < a.Cout) {
            const size_t kid = (size_t)co * CIN + ci;
            const unsigned m = smask[a.pid[kid]];
            size_t j = kid * a.k;
#pragma unroll
            for (int t = 0; t < 9; ++t)
                if (m & (1u << t)) wv[t] = load_val(a.val, j++, a.val_dtype);
        }
#pragma unroll
        for (int t = 0; t < 9; ++t) sWd[col][ci * 9 + t] = wv[t];
        if (ci == 0) {
            sWd[col][CIN * 9] = (a.bias && co < a.Cout) ? a.bias[co] : 0.f;
            for (int t = CIN * 9 + 1; t < KW; ++t) sWd[col][t] = 0.f;
        }
    }
    __syncthreads();

    const T* __restrict__ xg = reinterpret_cast<const T*>(a.x);
    T* __restrict__ yg = reinterpret_cast<T*>(a.y);
    const int Cs = a.y_c_stride;
    constexpr int PER16 = 16 / (int)sizeof(T);
    const bool vec = a.layout == RTOSS_NHWC && (Cs * sizeof(T)) % 16 == 0 && ((a.y_c_off + co0) * sizeof(T)) % 16 == 0 &&
                     co0 + kStemCo <= a.Cout;
    // 16-bit NHWC outputs whose rows hold whole groups: pixel index = kStemPx * group index + px, the pixels of a
    // round of the block are consecutive, and the stores go through the staging buffer
    const bool staged = sizeof(T) == 2 && vec && a.Wo % kStemPx == 0;
    const bool fast_in = sizeof(T) == 2 && CIN == 3 && S == 2 && kStemPx == 4 && a.layout == RTOSS_NHWC && a.W % 8 == 0;
    const int groups = (a.Wo + kStemPx - 1) / kStemPx;      // groups of kStemPx output columns per row
    const long long total = (long long)a.N * a.Ho * groups;
    const long long px_total = (long long)a.N * a.Ho * a.Wo;

    for (long long blk = blockIdx.x; blk * kStemThreads < total; blk += gridDim.x) {
        const long long gi_raw = blk * kStemThreads + threadIdx.x;
        const bool active = gi_raw < total;
        const long long gi = active ? gi_raw : total - 1;   // idle threads recompute the last group and store nothing
        const int ox0 = (int)(gi % groups) * kStemPx;
        const long long r1 = gi / groups;
        const int oy = (int)(r1 % a.Ho), n = (int)(r1 / a.Ho);
        float xin[CIN][3][WIN];
        if (fast_in) {
#pragma unroll
            for (int r = 0; r < 3; ++r) {
                const int iy = oy * S + r - 1;
                const bool row_ok = iy >= 0 && iy < a.H;
                // 16-byte piece 3 * (ox0 / 4) of the row holds input pixel 2 * ox0; the window starts one pixel earlier
                const uint4* rowp = reinterpret_cast<const uint4*>(xg + ((size_t)n * a.H + (row_ok ? iy : 0)) * a.W * CIN) + (ox0 / kStemPx) * 3;
                const uint4 zero = make_uint4(0u, 0u, 0u, 0u);
                uint4 ch[4];
                ch[0] = (row_ok && ox0 > 0) ? __ldg(rowp - 1) : zero;
#pragma unroll
                for (int i = 1; i < 4; ++i) ch[i] = row_ok ? __ldg(rowp + i - 1) : zero;
                const unsigned wds[16] = {ch[0].x, ch[0].y, ch[0].z, ch[0].w, ch[1].x, ch[1].y, ch[1].z, ch[1].w,
                                          ch[2].x, ch[2].y, ch[2].z, ch[2].w, ch[3].x, ch[3].y, ch[3].z, ch[3].w};
#pragma unroll
                for (int c = 0; c < WIN; ++c)
#pragma unroll
                    for (int ci = 0; ci < CIN; ++ci) {
                        const int hi = (5 + c * CIN + ci) & 31;   // 16-bit index inside the 64 bytes: the window starts at byte 10
                        const unsigned short bits = (hi & 1) ? (unsigned short)(wds[hi >> 1] >> 16) : (unsigned short)(wds[hi >> 1] & 0xFFFFu);
                        T v;
                        memcpy(&v, &bits, sizeof(bits));
                        xin[ci][r][c] = to_f32<T>(v);
                    }
            }
        } else {
#pragma unroll
            for (int r = 0; r < 3; ++r) {
                const int iy = oy * S + r - 1;
                const bool row_ok = iy >= 0 && iy < a.H;
#pragma unroll
                for (int c = 0; c < WIN; ++c) {
                    const int ix = ox0 * S + c - 1;
                    const bool ok = row_ok && ix >= 0 && ix < a.W;
#pragma unroll
                    for (int ci = 0; ci < CIN; ++ci) {
                        const size_t idx = a.layout == RTOSS_NCHW ? (((size_t)n * CIN + ci) * a.H + iy) * a.W + ix
                                                                  : (((size_t)n * a.H + iy) * a.W + ix) * CIN + ci;
                        xin[ci][r][c] = ok ? to_f32<T>(xg[idx]) : 0.f;
                    }
                }
            }
        }
        // kStemNf filters per trip of a loop that is NOT unrolled: with all 32 filters unrolled the body was 17 KB of
        // instructions and the warps waited for instruction fetch more than for anything else
#pragma unroll 1
        for (int q0 = 0; q0 < kStemCo; q0 += kStemNf) {
            __align__(8) T o[kStemPx][kStemNf];
#pragma unroll
            for (int q = 0; q < kStemNf; ++q) {
                float w[KW];
                const float4* wr = reinterpret_cast<const float4*>(sWd[q0 + q]);
#pragma unroll
                for (int i = 0; i < KW / 4; ++i) {
                    const float4 v = wr[i];
                    w[4 * i] = v.x;
                    w[4 * i + 1] = v.y;
                    w[4 * i + 2] = v.z;
                    w[4 * i + 3] = v.w;
                }
#pragma unroll
                for (int px = 0; px < kStemPx; ++px) {
                    float acc = w[CIN * 9];
#pragma unroll
                    for (int ci = 0; ci < CIN; ++ci)
#pragma unroll
                        for (int r = 0; r < 3; ++r)
#pragma unroll
                            for (int c = 0; c < 3; ++c) acc = fmaf(w[ci * 9 + r * 3 + c], xin[ci][r][px * S + c], acc);
                    o[px][q] = from_f32<T>(stem_act<T>(acc, a.act));
                }
            }
#pragma unroll
            for (int px = 0; px < kStemPx; ++px) {
                const int ox = ox0 + px;
                if (staged) {
                    // 8 bytes (four 16-bit filters) into the thread's 64 bytes of pixel px
                    reinterpret_cast<uint2*>(sOut)[(threadIdx.x * kStageRow + px * 4) * 2 + q0 / kStemNf] =
                        *reinterpret_cast<const uint2*>(o[px]);
                    continue;
                }
                if (ox >= a.Wo || !active) continue;
#pragma unroll
                for (int q = 0; q < kStemNf; ++q) {
                    const int co = co0 + q0 + q;
                    if (co < a.Cout) {
                        const size_t idx = a.layout == RTOSS_NCHW ? (((size_t)n * Cs + a.y_c_off + co) * a.Ho + oy) * a.Wo + ox
                                                                  : (((size_t)n * a.Ho + oy) * a.Wo + ox) * Cs + a.y_c_off + co;
                        yg[idx] = o[px][q];
                    }
                }
            }
        }
        if (staged) {
            __syncthreads();
            const long long px_first = blk * kStemThreads * kStemPx;   // first pixel of this round of the block
#pragma unroll 4
            for (int it = 0; it < kStemPx * 4; ++it) {
                const int q = it * kStemThreads + threadIdx.x;        // 16-byte piece of the round's outputs, in memory order
                const int pl = q >> 2, part = q & 3;                   // pixel inside the round, 8-filter group
                const long long pg = px_first + pl;
                if (pg < px_total)
                    *reinterpret_cast<uint4*>(yg + (size_t)pg * Cs + a.y_c_off + co0 + part * PER16) =
                        sOut[(pl / kStemPx) * kStageRow + (pl % kStemPx) * 4 + part];
            }
            __syncthreads();   // the staging buffer is free for the next round
        }
    }
}

template <typename T, int S>
int launch_small_cin_s(const Conv3Args& a, cudaStream_t stream) {
    const long long total = (long long)a.N * a.Ho * ((a.Wo + kStemPx - 1) / kStemPx);
    long long blocks = (total + kStemThreads - 1) / kStemThreads;
    if (blocks > 148 * 6) blocks = 148 * 6;   // a few rounds per block
    dim3 grid((unsigned)blocks, (unsigned)((a.Cout + kStemCo - 1) / kStemCo));
    switch (a.Cin) {
        case 1: rtoss_dev::launch_pdl(conv3x3_small_cin_kernel<T, 1, S>, grid, kStemThreads, 0, stream, a); break;
        case 2: rtoss_dev::launch_pdl(conv3x3_small_cin_kernel<T, 2, S>, grid, kStemThreads, 0, stream, a); break;
        case 3: rtoss_dev::launch_pdl(conv3x3_small_cin_kernel<T, 3, S>, grid, kStemThreads, 0, stream, a); break;
        default: rtoss_dev::launch_pdl(conv3x3_small_cin_kernel<T, 4, S>, grid, kStemThreads, 0, stream, a); break;
    }
    return (int)cudaGetLastError();
}

template <typename T>
int launch_small_cin(const Conv3Args& a, int stride, cudaStream_t stream) {
    return stride == 1 ? launch_small_cin_s<T, 1>(a, stream) : launch_small_cin_s<T, 2>(a, stream);
}

// Pick the lane arrangement that wastes the fewest lanes and pixels.
void choose_lanes(int Ho, int Wo, int PH, int PW, int S, int* LX, int* LY) {
    double best = -1.0;
    for (int lx = 1; lx <= 16; ++lx)
        for (int ly = 1; ly * lx <= 32; ++ly) {
            const int tw = lx * PW, th = ly * PH;
            const double cover = (double)((Wo + tw - 1) / tw * tw) * ((Ho + th - 1) / th * th);
            double util = (double)Wo * Ho / cover * (lx * ly) / 32.0;
            // staging cost grows with the halo: staged input pixels per output pixel
            util /= 1.0 + 0.25 * ((double)((tw * S + 2) * (th * S + 2)) / (double)(tw * th * S * S) - 1.0);
            if (util > best) {
                best = util;
                *LX = lx;
                *LY = ly;
            }
        }
}

inline int round_up(int v, int m) { return (v + m - 1) / m * m; }

// Tiling and staging plan of one call for a kernel shape (PH x PW output pixels per lane, CO_T filters per warp, WARPS
// warps, MINB CTAs per SM): lane arrangement, tile sizes, how the activations travel, shared-memory layout.  Host
// arithmetic only.  Returns the dynamic shared memory in bytes, or 0 when the shape does not fit.
//
// NCHW activations travel as aligned vectors of vb bytes through cp.async.  A vector's address is
//   base + ((n*Cin + ci)*H*W + iy*W + ox0*S - veq + j*veq) * es,   ox0 = tx * LX * PW,  veq = vb / es,
// so vb has to divide the row pitch W*es AND the byte step between neighbouring tiles, LX*PW*S*es: with four pixels per
// lane and an odd number of lane columns every second tile of a 16-bit image starts 8 bytes off a 16-byte boundary
// (a misaligned-address fault on a 64-channel 40x40 bf16 layer once showed exactly that).
size_t plan_variant(Conv3Args& a, int es, int S, int PH, int PW, int CO_T, int WARPS, int MINB) {
    const int CO_BLOCK = WARPS * CO_T;
    choose_lanes(a.Ho, a.Wo, PH, PW, S, &a.LX, &a.LY);
    a.tiles_x = (a.Wo + a.LX * PW - 1) / (a.LX * PW);
    a.tiles_y = (a.Ho + a.LY * PH - 1) / (a.LY * PH);
    a.TW_in = (a.LX * PW - 1) * S + 3;
    a.TH_in = (a.LY * PH - 1) * S + 3;
    a.TWP = round_up(a.TW_in, 4);
    a.plane = round_up(a.TH_in * a.TWP, 32) + 4;

    a.w_async = (a.Cin % 8 == 0) ? 1 : 0;
    a.rawV_bytes = a.w_async ? CO_BLOCK * 8 * a.k * a.val_esize : 0;
    const int fixed_bytes = (int)sizeof(float) * kCiChunk * (a.plane + CO_BLOCK * kWSlots) + 2 * a.rawV_bytes +
                            (a.w_async ? 2 * CO_BLOCK * 8 : 0);
    const int smem_cap = (MINB > 1 ? 227 * 1024 / MINB - 1024 : 200 * 1024);  // leave room for MINB CTAs per SM

    // how the activations travel: cp.async where rows are aligned and the raw buffers fit, else plain loads
    a.xmode = X_SYNC;
    a.vb = 0;
    a.EV = 0;
    int n_tab = a.TH_in * a.TWP;
    a.rawX_bytes = 0;
    const bool x16 = (reinterpret_cast<uintptr_t>(a.x) & 15) == 0;
    if (a.layout == RTOSS_NCHW && x16) {
        const int row_bytes = a.W * es, step_bytes = a.LX * PW * S * es;
        int vb = 0;
        for (int cand = 16; cand >= 4 && !vb; cand >>= 1)
            if (row_bytes % cand == 0 && step_bytes % cand == 0) vb = cand;
        if (vb >= es && vb > 0) {
            const int veq = vb / es;
            const int nv = round_up(veq - 1 + a.TW_in, veq) / veq;
            const int raw = round_up(kCiChunk * a.TH_in * nv * vb, 16);
            if (fixed_bytes + 2 * raw + 8 * a.TH_in * nv <= smem_cap) {
                a.xmode = X_NCHW_VEC;
                a.vb = vb;
                a.EV = a.TH_in * nv;
                n_tab = a.EV;
                a.rawX_bytes = raw;
            }
        }
    } else if (a.layout == RTOSS_NHWC && x16 && a.Cin % 8 == 0) {
        const int raw = round_up(a.TH_in * a.TW_in * 8 * es, 16);
        if (fixed_bytes + 2 * raw + 8 * a.TH_in * a.TW_in <= smem_cap) {
            a.xmode = X_NHWC_VEC;
            a.vb = 16;
            a.EV = a.TH_in * a.TW_in;
            n_tab = a.EV;
            a.rawX_bytes = raw;
        }
    }

    int off = (int)sizeof(float) * kCiChunk * a.plane;
    a.off_sW = off;
    off += (int)sizeof(float) * kCiChunk * CO_BLOCK * kWSlots;
    a.off_rawX = off;
    off += 2 * a.rawX_bytes;
    a.off_rawV = off;
    off += 2 * a.rawV_bytes;
    a.off_rawP = off;
    off += a.w_async ? 2 * CO_BLOCK * 8 : 0;
    a.off_tab = off;
    off += 2 * (int)sizeof(int) * n_tab;
    return off > 220 * 1024 ? 0 : (size_t)off;
}

template <typename T, int S, int PH, int PW, int CO_T, int WARPS, int MINB>
int launch_variant(Conv3Args& a, cudaStream_t stream) {
    constexpr int CO_BLOCK = WARPS * CO_T;
    constexpr int kThreads = WARPS * 32;
    const size_t smem = plan_variant(a, (int)sizeof(T), S, PH, PW, CO_T, WARPS, MINB);
    if (!smem) return (int)cudaErrorInvalidConfiguration;
    auto kern = conv3x3_alu_kernel<T, S, PH, PW, CO_T, WARPS, MINB>;
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return (int)e;
    dim3 grid((unsigned)((size_t)a.tiles_x * a.tiles_y * a.N), (unsigned)((a.Cout + CO_BLOCK - 1) / CO_BLOCK));
    rtoss_dev::launch_pdl(kern, grid, kThreads, smem, stream, a);
    return (int)cudaGetLastError();
}

// Which kernel shape takes a call: one output row of eight pixels per lane, eight filters per warp, eight warps, two
// CTAs per SM; a layer that fills fewer than half the SMs that way takes the finer shape (four pixels per lane, four
// filters per warp, four warps, four CTAs per SM: a quarter of the outputs per CTA).
struct FmaShape {
    int PH, PW, CO_T, WARPS, MINB;
};
FmaShape choose_shape(const Conv3Args& a0, int es, int S) {
    Conv3Args a = a0;
    const FmaShape big = {1, 8, 8, 8, 2}, fine = {1, 4, 4, 4, 4};
    if (!plan_variant(a, es, S, big.PH, big.PW, big.CO_T, big.WARPS, big.MINB)) return big;
    const long ctas = (long)a.tiles_x * a.tiles_y * a.N * ((a.Cout + 63) / 64);
    return ctas < 74 ? fine : big;
}

template <typename T>
int launch_typed(Conv3Args& a, int stride, cudaStream_t stream) {
    if (a.Cin <= 4) return launch_small_cin<T>(a, stride, stream);
    const FmaShape sh = choose_shape(a, (int)sizeof(T), stride);
    if (sh.PW == 4) {
        if (stride == 1) return launch_variant<T, 1, 1, 4, 4, 4, 4>(a, stream);
        return launch_variant<T, 2, 1, 4, 4, 4, 4>(a, stream);
    }
    if (stride == 1) return launch_variant<T, 1, 1, 8, 8, 8, 2>(a, stream);
    return launch_variant<T, 2, 1, 8, 8, 8, 2>(a, stream);
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
    a.val_esize = (int)rtoss_dtype_size(p->dtype);
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

// The tiling the FMA path would use for a 3x3 call (host arithmetic only; see rtoss.h).
extern "C" rtoss_status rtoss_fma_plan3x3(const rtoss_conv_desc* d, int Cin, int Cout, int k, rtoss_dtype packed_dtype,
                                          rtoss_fma_plan* out) {
    if (!d || !out || Cin < 1 || Cout < 1 || k < 1 || k > 9 || d->N < 1 || d->H < 1 || d->W < 1 || (d->stride != 1 && d->stride != 2) ||
        (int)d->io_dtype < 0 || (int)d->io_dtype > 2 || (int)packed_dtype < 0 || (int)packed_dtype > 2)
        return RTOSS_ERR_INVALID_ARG;
    memset(out, 0, sizeof(*out));
    if (Cin <= 4) {
        out->small_cin = 1;   // the kernel for up to four input channels: no staging plan
        return RTOSS_OK;
    }
    Conv3Args a;
    memset(&a, 0, sizeof(a));
    a.x = nullptr;   // (a 16-byte aligned pointer)
    a.val_dtype = (int)packed_dtype;
    a.val_esize = (int)rtoss_dtype_size(packed_dtype);
    a.N = d->N;
    a.Cin = Cin;
    a.Cout = Cout;
    a.H = d->H;
    a.W = d->W;
    a.Ho = (d->H - 1) / d->stride + 1;
    a.Wo = (d->W - 1) / d->stride + 1;
    a.k = k;
    a.layout = (int)d->layout;
    const int es = (int)rtoss_dtype_size(d->io_dtype);
    const FmaShape sh = choose_shape(a, es, d->stride);
    const size_t smem = plan_variant(a, es, d->stride, sh.PH, sh.PW, sh.CO_T, sh.WARPS, sh.MINB);
    if (!smem) return RTOSS_ERR_UNSUPPORTED;
    out->pixels_per_lane = sh.PW;
    out->filters_per_warp = sh.CO_T;
    out->warps = sh.WARPS;
    out->ctas_per_sm = sh.MINB;
    out->lanes_x = a.LX;
    out->lanes_y = a.LY;
    out->tiles_x = a.tiles_x;
    out->tiles_y = a.tiles_y;
    out->grid_x = a.tiles_x * a.tiles_y * a.N;
    out->grid_y = (Cout + sh.WARPS * sh.CO_T - 1) / (sh.WARPS * sh.CO_T);
    out->staged_rows = a.TH_in;
    out->staged_cols = a.TW_in;
    out->staging = a.xmode;
    out->vector_bytes = a.vb;
    out->vectors_per_plane = a.EV;
    out->shared_bytes = (int)smem;
    return RTOSS_OK;
}
