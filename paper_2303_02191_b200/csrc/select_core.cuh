// Per-kernel arithmetic of pattern selection and packing (Algorithm 2; Algorithm 3 after regrouping), shared by
// the single-layer kernels and the whole-model batch so that both give the same bits.
#ifndef RTOSS_SELECT_CORE_CUH
#define RTOSS_SELECT_CORE_CUH

#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>

#include <cstdint>

namespace rtoss_dev {

// Squares in fp32, pattern sums in fp32 over ascending taps, first strictly larger sum wins (ties -> lowest id,
// a NaN sum never wins).  __fmul_rn / __fadd_rn keep the compiler from contracting or reordering the arithmetic.
// `tab[p]` is the 9-bit mask of pattern p.
template <typename Tab>
__device__ __forceinline__ int select_best(const float (&w)[9], const Tab& tab, int P) {
    float q[9];
#pragma unroll
    for (int t = 0; t < 9; ++t) q[t] = __fmul_rn(w[t], w[t]);
    int best = 0;
    float best_s = 0.f;
    for (int p = 0; p < P; ++p) {
        const unsigned m = tab[p];
        float s = 0.f;
#pragma unroll
        for (int t = 0; t < 9; ++t)
            if (m & (1u << t)) s = __fadd_rn(s, q[t]);
        if (p == 0) {
            best_s = s;
        } else if (s > best_s || (best_s != best_s && s == s)) {
            best = p;
            best_s = s;
        }
    }
    return best;
}

template <typename V> __device__ __forceinline__ V narrow_to(float v);
template <> __device__ __forceinline__ float narrow_to<float>(float v) { return v; }
template <> __device__ __forceinline__ __nv_bfloat16 narrow_to<__nv_bfloat16>(float v) { return __float2bfloat16_rn(v); }
template <> __device__ __forceinline__ __half narrow_to<__half>(float v) { return __float2half_rn(v); }

// Writes of one kernel (3x3) or run of nine (1x1) with mask m: its k kept values, ascending taps, rounded to V, to
// val[i*k ...]; and, where the handle carries dense-expanded weights for the tensor path (wtc != nullptr), all nine
// taps, pruned ones as +0:  3x3 -> wtc[t][row][ci] with `rows` rows per tap, filter co = i / Cin at rows
// c*rep_rows + co for c < copies (one copy at row co in the plain layout);  1x1 -> wtc[9*i + t].  fp32 handles hold
// two such arrays back to back: tf32 heads, then remainders.
template <typename V>
__device__ __forceinline__ void pack_one(const float (&w)[9], unsigned m, int64_t i, int k, V* __restrict__ val,
                                         V* __restrict__ wtc, int ksize, int Cin, int rows, int rep_rows, int copies) {
    V* out = val + i * k;
    if (k * (int)sizeof(V) == 8) {
        // the k kept values of a kernel are 8 aligned bytes (four 16-bit or two 32-bit values): pushed into a 64-bit word
        // from the top, tap by tap in ascending order, so that after k pushes the first kept value sits in the lowest
        // bits (a valid mask has exactly k bits); written with one store
        unsigned long long word = 0;
#pragma unroll
        for (int t = 0; t < 9; ++t) {
            if (m & (1u << t)) {
                const V v = narrow_to<V>(w[t]);
                unsigned long long bits;
                if constexpr (sizeof(V) == 4) {
                    bits = (unsigned long long)__float_as_uint(v);
                } else {
                    bits = (unsigned long long)*reinterpret_cast<const unsigned short*>(&v);
                }
                word = (word >> (8 * sizeof(V))) | (bits << (64 - 8 * sizeof(V)));
            }
        }
        *reinterpret_cast<unsigned long long*>(out) = word;
    } else {
        int j = 0;
#pragma unroll
        for (int t = 0; t < 9; ++t)
            if (m & (1u << t)) out[j++] = narrow_to<V>(w[t]);
    }
    if (wtc) {
        // (layers hold fewer than 2^31 kernels: 32-bit division, several times cheaper than the 64-bit one)
        const int64_t co = (int64_t)((unsigned)i / (unsigned)Cin), ci = i - co * Cin;
        // fp32: the tensor path multiplies tf32 operands, so every weight is stored as its tf32 head (the 19 leading bits)
        // and, in a second copy of the array behind the first, the remainder (exact in fp32)
        const int64_t lo_at = (int64_t)(ksize == 3 ? 9 : 1) * rows * Cin;
#pragma unroll
        for (int t = 0; t < 9; ++t) {
            V v = (m & (1u << t)) ? narrow_to<V>(w[t]) : narrow_to<V>(0.f);
            V lo = v;
            if (sizeof(V) == 4) {
                const float f = (m & (1u << t)) ? w[t] : 0.f;
                const float head = __uint_as_float(__float_as_uint(f) & 0xFFFFE000u);
                v = narrow_to<V>(head);
                lo = narrow_to<V>(__fsub_rn(f, head));
            }
            if (ksize == 3) {
                const int64_t at = ((int64_t)t * rows + co) * Cin + ci;   // copy 0; copy c lies c * rep_rows rows further down
                for (int c = 0; c < copies; ++c) {
                    wtc[at + (int64_t)c * rep_rows * Cin] = v;
                    if (sizeof(V) == 4) wtc[lo_at + at + (int64_t)c * rep_rows * Cin] = lo;
                }
            } else {
                wtc[i * 9 + t] = v;
                if (sizeof(V) == 4) wtc[lo_at + i * 9 + t] = lo;
            }
        }
    }
}

// Stable counting sort of the Cout filters of input channel ci by pattern id, by one warp: perm[ci*Cout + j] lists
// the filters by ascending id (ties by ascending filter), bucket_off[ci*(P+1) + p] is where pattern p starts.
// Ranks inside a group of 32 filters come from __match_any_sync; `fill` is 256 words of shared memory of this warp.
// Ids must be < P; a filter whose id is not is left out of perm (the channel's list is then short by it, the last
// bucket ends before bucket_off's closing entry Cout) rather than written past the channel's slice.
//
// On the way the warp also records which taps the tensor path has to multiply at all: `issue` (nullable) holds one
// 64-bit word per (tile of 128 filters, block of 2^cb_log2 input channels: 64 for 16-bit handles, 32 for fp32 ones --
// 128 bytes of a row), bit 4 t + s set when some kernel of the tile with its channel in slab s (a quarter) of the
// block keeps tap t (the union of the kept taps over the tile, from
// `masks`, the table as the device sees it).  The words must be zero before the pass; channels add their bits with
// atomicOr.  A (tile, slab, tap) whose bit stays clear holds only pruned weights: its matrix instruction is skipped.
__device__ __forceinline__ void order_channel(const uint8_t* __restrict__ pid, int Cout, int Cin, int P, int ci,
                                              uint32_t* __restrict__ perm, uint32_t* __restrict__ bucket_off,
                                              uint32_t* fill, int lane, const uint16_t* __restrict__ masks = nullptr,
                                              unsigned long long* __restrict__ issue = nullptr, int cb_log2 = 6) {
    for (int p = lane; p < 256; p += 32) fill[p] = 0;
    __syncwarp();
    // pass 1: histogram
    unsigned used = 0;   // taps kept by any filter of the current tile of 128
    const int cb_mask = (1 << cb_log2) - 1, ncb = (Cin + cb_mask) >> cb_log2;
    for (int base = 0; base < Cout; base += 32) {
        const int co = base + lane;
        unsigned key = co < Cout ? pid[(size_t)co * Cin + ci] : 0xFFFFu;
        if (key >= (unsigned)P) key = 0xFFFFu;   // an id outside the table is not placed (nothing is written for it)
        const unsigned peers = __match_any_sync(0xFFFFFFFFu, key);
        if (key != 0xFFFFu && lane == __ffs(peers) - 1) fill[key] += __popc(peers);
        if (issue) {
            used |= __reduce_or_sync(0xFFFFFFFFu, key != 0xFFFFu ? (unsigned)masks[key] : 0u);
            if (((base + 32) & 127) == 0 || base + 32 >= Cout) {
                if (lane == 0 && used) {
                    unsigned long long bits = 0;
#pragma unroll
                    for (int t = 0; t < 9; ++t)
                        if (used & (1u << t)) bits |= 1ull << (4 * t + ((ci & cb_mask) >> (cb_log2 - 2)));
                    atomicOr(issue + (size_t)(base >> 7) * ncb + (ci >> cb_log2), bits);
                }
                used = 0;
            }
        }
        __syncwarp();
    }
    // exclusive scan over the P buckets (P <= 255: eight per lane, then a warp scan of lane totals)
    uint32_t local[8];
    uint32_t sum = 0;
#pragma unroll
    for (int j = 0; j < 8; ++j) {
        const int p = lane * 8 + j;
        local[j] = sum;
        sum += (p < P) ? fill[p] : 0;
    }
    uint32_t incl = sum;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
        uint32_t o = __shfl_up_sync(0xFFFFFFFFu, incl, d);
        if (lane >= d) incl += o;
    }
    const uint32_t excl = incl - sum;
    __syncwarp();
#pragma unroll
    for (int j = 0; j < 8; ++j) {
        const int p = lane * 8 + j;
        if (p < P) {
            fill[p] = excl + local[j];
            bucket_off[(size_t)ci * (P + 1) + p] = excl + local[j];
        }
    }
    if (lane == 0) bucket_off[(size_t)ci * (P + 1) + P] = (uint32_t)Cout;
    __syncwarp();
    // pass 2: placement, filters in ascending order inside each bucket
    for (int base = 0; base < Cout; base += 32) {
        const int co = base + lane;
        unsigned key = co < Cout ? pid[(size_t)co * Cin + ci] : 0xFFFFu;
        if (key >= (unsigned)P) key = 0xFFFFu;
        const unsigned peers = __match_any_sync(0xFFFFFFFFu, key);
        const unsigned before = peers & ((1u << lane) - 1u);
        if (key != 0xFFFFu) perm[(size_t)ci * Cout + fill[key] + __popc(before)] = (uint32_t)co;
        __syncwarp();
        if (key != 0xFFFFu && before == 0) fill[key] += __popc(peers);
        __syncwarp();
    }
}

}  // namespace rtoss_dev

#endif
