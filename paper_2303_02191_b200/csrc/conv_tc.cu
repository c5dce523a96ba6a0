// Tensor-core path of the pattern convolutions (bf16 / fp16, NHWC, stride 1 or 2).
//
// Per-kernel patterns cannot be compacted into a dense contraction (every
// filter keeps different (channel, tap) positions), so this path evaluates the
// convolution of Section II.B of arXiv 2303.02191 as a masked dense implicit
// GEMM on the 5th-generation tensor cores: the pruned taps are multiplied as
// zeros.  It performs 9/k times the non-zero FLOPs and is still several times
// faster than the FMA-pipe gather for 16-bit data; the FMA path stays the one
// for fp32 and for shapes this kernel does not take.
//
// GEMM view:  D[co, position] = sum over taps t and channels ci of
//                               Wt[t][co][ci] * X[position shifted by t, ci]
//   * A CTA tile is TH output rows of one image (all columns) times 128 output
//     channels.  The input rows it needs (with the one-pixel halo, zero-filled
//     by TMA outside the image) are staged once per block of 64 channels as a
//     flat list of "padded pixels", 128 bytes (64 channels) each, row pitch
//     Wp = W + 2 pixels.  In that list the input pixel of tap (r, c) for output
//     position p is at p + r*Wp + c: the activation operand of every tap is
//     the SAME shared-memory tile read from a different start row, so the halo
//     tile is loaded once and used by all nine taps.  Output positions run over
//     the padded pitch too; the two junk positions per row are computed and
//     dropped.
//   * Operand roles: the weights are the M operand (128 filters = the 128 TMEM
//     lanes), the positions are the N operand (up to 256 per instruction), K =
//     16 channels per instruction.  One instruction costs about 140 cycles
//     whatever N is, and with M = 64 as with M = 128 (measured), so N
//     must be wide: 128 x 256 x 16 per instruction runs near the tensor peak,
//     128 x 128 x 16 at half of it (measured on this kernel with both roles).
//   * Weights are the dense-expanded form Wt[t][co][ci] that rtoss_pack builds
//     next to the packed arrays; one TMA box per (kernel row of three taps,
//     channel block); filters
//     beyond Cout are zero-filled by TMA.
//   * Persistent CTAs, one per SM, each walking a strided list of tiles.  Warp
//     roles: warp 0 issues the TMA copies of the activations, warp 1 issues
//     tcgen05.mma and owns the TMEM allocation, warps 2..17 run the epilogue
//     (tcgen05.ld, bias, activation, rounding, a transpose through shared memory,
//     16-byte NHWC stores), warp 18 issues the TMA copies of the weights (a stage
//     of three taps is one copy: issuing a copy occupies its thread for hundreds
//     of cycles whatever the size).  Activation and weight stages form rings
//     that run on across tiles; two accumulator stages in TMEM let the epilogue
//     of a tile run under the MMAs of the next.
//   * Layers with few tiles and long channel loops are cut along the channel
//     blocks: the CTAs that share a tile form a thread-block cluster and exchange
//     their partial sums through distributed shared memory (split K).
//   * Launched with programmatic stream serialization: barrier set-up, TMEM allocation and descriptor
//     prefetch run before griddepcontrol.wait, i.e. possibly under the tail of the previous kernel.
//   * Every mbarrier wait is bounded; a wait that runs out records a code in
//     the context's status word and the CTA leaves through the normal exit
//     (TMEM is always released).
//   * A 3x3 layer's handle says, per (tile of 128 filters, 16-channel slab, tap), whether any kept weight lies there
//     (rtoss_pack gathers that from the pattern ids).  Where none does, the instruction would multiply zeros only and
//     is not issued.  With per-kernel patterns on dense random weights every such block holds kept weights; when a
//     block of kernels shares one pattern (rtoss_select_patterns_shared) only k of the 9 taps of a slab are issued:
//     the contraction is then compacted to the non-zero work.
//   * fp32 data runs on the same pipeline with kind::tf32 instructions and three products per tap in place of one:
//     every value is split into a tf32 head (19 leading bits) and the remainder, x = xh + xl, w = wh + wl, and
//     wh*xh + wh*xl + wl*xh is accumulated in fp32 (the dropped wl*xl is below 2^-21 of the product).  The weights are
//     split when they are packed; an activation block is split in shared memory by the warp that fetched it (head in
//     place, remainder into the second half of the stage) before the MMA thread may read it.
//   * One launch may carry several independent convolutions ("problems": the pyramid levels of a detection tower,
//     the two branches of a block): the tile list runs over all of them, every role looks its tile's problem up.
//     Small problems then fill the tail of the large ones' waves instead of paying a launch each.
#include <cuda.h>
#include <cudaTypedefs.h>

#include <atomic>
#include <cstring>
#include <utility>

#include "conv_common.cuh"

namespace {

using namespace rtoss_dev;

constexpr int kEpiWarps = 16;
constexpr int kTcThreads = (3 + kEpiWarps) * 32;  // activation TMA warp, MMA warp, sixteen epilogue warps, weight TMA warp
constexpr int kWeightWarp = 2 + kEpiWarps;        // the last warp loads the weights
constexpr int kPatchRows = 16;       // positions an epilogue warp turns at a time
constexpr int kMaxA = 4, kMaxB = 8;  // most activation stages / weight slots
constexpr int kMTile = 128;          // filters per tile = TMEM lanes
constexpr int kPxmMaxCout = 64;      // layers this narrow run with positions as the M operand
constexpr int kMaxPx = 256;          // most positions in a tile's list
constexpr int kPairPitch = 144;      // bytes per row (a pair of positions x 32 filters, + 16 pad) of the packed patch
constexpr int kResStage = 2048;   // per epilogue warp: two buffers of 2 x 32 residual pieces of 16 bytes
constexpr int kPatchBytes = kPatchRows / 2 * kPairPitch;  // an epilogue warp's transpose patch
constexpr int kKBlock = 64;       // channels per staged block: 128 bytes of bf16 / fp16
constexpr int kRowBytes = 128;    // one padded pixel, one channel block
constexpr long long kWaitCycles = 2000000000LL;  // about one second

constexpr int kMaxProb = 20;      // convolutions one launch may carry
constexpr int kMaxTabs = 8;       // distinct position tables of a launch (problems of equal tile geometry share one)

// One convolution of a launch.
struct TcArgs {
    void* y;
    const void* resid;   // residual operand laid out like y, or null
    int resid_post;      // 1: the residual is added behind the activation (y = act(conv) + residual), 0: in front of it
    const float* bias;
    const unsigned long long* issue;   // 3x3: which (tap, slab) pairs of (filter tile, channel block) to multiply; null = all
    int N, Ho, Wo, Cin, Cout;    // output image size
    int S;                       // stride
    int Wq, TH, TW, taps;        // position pitch, output rows and columns per tile, 9 or 1
    int N_px, ncb;               // positions per tile (the MMA's N, multiple of 16), channel blocks
    int tiles_y, tiles_x, co_tiles;
    // A unit's index is taken apart into (share of the channel blocks, filter tile, column segment, row band, image) by
    // every role for every tile: the four divisors as multiply-and-shift pairs (see tile_of), set by the host.
    unsigned div_ks[2], div_co[2], div_tx[2], div_ty[2];
    int n_sub, sub_bytes;        // staged sub-tiles per channel block (4 input phases for 3x3 stride 2) and their size
    int x_add[4], y_add[4];      // TMA start coordinate of sub-tile s: x = x0*S + x_add[s], y = y0*S + y_add[s]
    int tap_sub[9], tap_shift[9];  // which sub-tile tap t reads, and from which start row
    int G;                                     // taps per weight stage (one barrier round trip per G taps)
    unsigned a_tx_bytes, b_tx_bytes;
    int act, y_c_off, y_c_stride, is_bf16;
    unsigned idesc;
    int w_rows;           // filter rows per staged weight tile (128; fewer with positions as the M operand)
    int rep_rows, R;      // filters as M, narrow layer: the tile holds R copies of rep_rows filter rows (else 128, 1)
    int rep_shift;        // log2(rep_rows)
    int pxm, MH, n_cols;  // positions as the M operand: M halves of 128 positions per tile, filters per tile (the MMA's N)
    // Split K: a tile's channel blocks are shared out to the KS CTAs of a thread-block cluster, cb_per blocks each;
    // the partial sums are exchanged through distributed shared memory and every CTA finishes a part of the tile.
    int KS, cb_per;
    int cb_ch, slab_ch;   // channels per staged block (128 bytes) and per instruction (32 bytes): 64 / 16 for 16-bit data, 32 / 8 for fp32
    // Bytes of a staged row (one padded pixel resp. one filter, one channel block): 128 with the 128-byte swizzle, or 64
    // with the 64-byte swizzle for 16-bit layers of at most 32 input channels (half of a 128-byte row would be zero fill,
    // and it is the traffic from L2 to shared memory that bounds such layers).  desc_hi: the matching upper word of the
    // shared-memory matrix descriptors.
    int row_bytes;
    unsigned desc_hi;
    int taps_real;        // 9 or 1; `taps` counts weight tiles per channel block: twice that for fp32 (heads, then remainders)
    int lo_off;           // fp32: byte offset of the remainders inside an activation stage
    // The operand rings this problem runs with: NA activation stages of a_stage bytes from the start of the ring area, NB
    // weight stages of b_stage bytes from sB_off.  Problems of one launch with the same `geo` share all five; where a
    // CTA passes to a problem of another geometry its rings run empty first (see bar_switch in the kernel).
    int NA, NB;
    unsigned a_stage, b_stage, sB_off;
    int geo;
    int tab;              // which of the launch's position tables
    // over_res: this problem's rings reach into the launch's residual staging area (only problems without a residual
    // operand may): a CTA that comes to it from a problem with one waits for that problem's epilogues first.
    int over_res;
    // Dependent problems of one launch: bit j of dep_mask = problem j (earlier in the launch's order) must be complete
    // -- all its outputs written -- before this one reads an activation or writes an output; done_target = arrivals
    // on this problem's counter that make it complete (epilogue warps x CTAs that hold units of it).
    unsigned dep_mask, done_target;
};

// A launch: up to NP convolutions sharing the CTA's rings (stage sizes are the largest any of them needs).  The struct
// travels as the kernel's parameter: a launch of one convolution carries the small instantiation (a large parameter
// block costs launch time).
template <int NP>
struct TcLaunchT {
    int n_prob;
    int unit_end[NP];   // units (tile x share of the channel blocks) of problems 0..i
    int* status;
    long long wait_cycles;    // limit of every wait
    int inject;               // test hook: 1 = the first weight copy of the launch is withheld (the wait for it must run out)
    int ring_bytes;           // the ring area: the most any problem's activation + weight stages take
    int max_na, max_nb;       // most activation / weight stages any problem uses (barriers to set up)
    int n_tabs;               // position tables
    int res_off;              // where in the ring area the staging of residual operands lies (its top end), when a problem has one
    unsigned* done;           // dependent problems: kMaxProb completion counters + one exit counter, all zero between launches; else null
    int AS, acc_stride;                        // accumulator stages in TMEM and columns per stage
    int tmem_cols;
    TcArgs prob[NP];
    CUtensorMap tmA[NP], tmB[NP];
};
using TcLaunch1 = TcLaunchT<1>;
using TcLaunchN = TcLaunchT<kMaxProb>;
static_assert(sizeof(TcLaunchN) <= 16384, "kernel parameters: well inside the 32 KB a launch may carry");
static_assert(kMaxProb <= 32, "dependencies are a 32-bit mask");

__device__ __forceinline__ unsigned smem_u32(const void* p) { return (unsigned)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(unsigned bar, unsigned count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(unsigned bar, unsigned bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
// Bounded wait on a phase parity; false when the limit ran out.
__device__ __forceinline__ unsigned mbar_try(unsigned bar, unsigned parity) {
    unsigned done;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(done)
        : "r"(bar), "r"(parity)
        : "memory");
    return done;
}
__device__ __forceinline__ bool mbar_wait(unsigned bar, unsigned parity, long long limit) {
    if (mbar_try(bar, parity)) return true;  // the common case costs one instruction, no clock read
    const long long t0 = clock64();
    for (;;) {
        if (mbar_try(bar, parity)) return true;
        if (clock64() - t0 > limit) return false;
    }
}

// Thread-block cluster primitives (split K): rank of this CTA, the address of a peer's shared memory, a store to it,
// and the cluster-wide barrier (release / acquire: stores to peers before it are visible after it).
__device__ __forceinline__ unsigned cluster_rank() {
    unsigned r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
__device__ __forceinline__ unsigned peer_smem(unsigned local_addr, unsigned rank) {
    unsigned r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(local_addr), "r"(rank));
    return r;
}
__device__ __forceinline__ void st_peer_f32(unsigned addr, float v) {
    asm volatile("st.shared::cluster.f32 [%0], %1;" ::"r"(addr), "f"(v) : "memory");
}
__device__ __forceinline__ void cluster_sync_all() {
    asm volatile("barrier.cluster.arrive.release;" ::: "memory");
    asm volatile("barrier.cluster.wait.acquire;" ::: "memory");
}

__device__ __forceinline__ void tma_load_4d(unsigned dst, const CUtensorMap* map, int c0, int c1, int c2, int c3,
                                            unsigned bar) {
    asm volatile(
        "cp.async.bulk.tensor.4d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4, %5}], [%6];"
        ::"r"(dst), "l"(map), "r"(c0), "r"(c1), "r"(c2), "r"(c3), "r"(bar)
        : "memory");
}
__device__ __forceinline__ void tma_load_3d(unsigned dst, const CUtensorMap* map, int c0, int c1, int c2, unsigned bar) {
    asm volatile(
        "cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];"
        ::"r"(dst), "l"(map), "r"(c0), "r"(c1), "r"(c2), "r"(bar)
        : "memory");
}

// Shared-memory matrix descriptor, K-major operand with 128-byte swizzle: rows of 128 bytes, groups
// of 8 rows 1024 bytes apart.  The start may be any 16-byte aligned address inside a tile whose base
// is 1024-byte aligned: the swizzle is a function of the absolute shared-memory address, the same
// function TMA applied when it wrote the tile, so a start in the middle of an 8-row group (a tap
// shift) or 32 bytes into a row (a K step) needs no correction (base-offset field 0).
// With rows of 64 bytes and the 64-byte swizzle the same holds for groups of 8 rows 512 bytes apart.
__host__ __device__ __forceinline__ unsigned long long make_sw_desc(unsigned addr, int row_bytes) {
    unsigned long long d = 0;
    d |= (unsigned long long)((addr & 0x3FFFFu) >> 4);        // start address
    d |= (unsigned long long)1 << 16;                          // leading byte offset (unused for swizzled K-major)
    d |= (unsigned long long)((8 * row_bytes) >> 4) << 32;     // stride byte offset: 8 rows
    d |= (unsigned long long)1 << 46;                          // descriptor version of this architecture
    d |= (unsigned long long)(row_bytes == 64 ? 4 : 2) << 61;  // 64-byte resp. 128-byte swizzle
    return d;
}

template <bool TF32>
__device__ __forceinline__ void umma_f16(unsigned d_tmem, unsigned long long adesc, unsigned long long bdesc,
                                         unsigned idesc, unsigned accumulate) {
    if (TF32)
        asm volatile(
            "{\n\t.reg .pred p;\n\t"
            "setp.ne.b32 p, %4, 0;\n\t"
            "tcgen05.mma.cta_group::1.kind::tf32 [%0], %1, %2, %3, p;\n\t}"
            ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
            : "memory");
    else
        asm volatile(
            "{\n\t.reg .pred p;\n\t"
            "setp.ne.b32 p, %4, 0;\n\t"
            "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
            ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
            : "memory");
}
// The MMAs of one tap of one channel block (filters on M) for the 16-channel slabs named by the mask m4 (bit s = slab
// s), with a look at the "full" barriers of the NEXT activation and weight stage started in front of them
// (mbarrier.test_wait: the answer comes back while the MMAs are being issued).  A wait costs the issuing thread a
// round trip of a few hundred cycles through a memory pipe the epilogue warps keep busy, and with four MMAs per wait
// nothing hides two of those per channel block; the stages ahead are normally full already, so the look usually
// replaces both waits of the next block.  The first instruction issued takes `accumulate` as its accumulate flag,
// the later ones add.  Returns bit 0: next activation stage full, bit 1: next weight stage full.
#define RTOSS_DEFINE_PEEK(NAME, KIND)                                                                                   \
    __device__ __forceinline__ unsigned NAME(unsigned d_tmem, unsigned long long adesc, unsigned long long bdesc,     \
                                             unsigned idesc, unsigned accumulate, unsigned m4, unsigned barA,          \
                                             unsigned parA, unsigned barB, unsigned parB) {                            \
        unsigned res;                                                                                                  \
        asm volatile(                                                                                                  \
            "{\n\t.reg .pred pa, pb, q, p0, p1, p2, p3;\n\t.reg .b64 a1, a2, a3, b1, b2, b3;\n\t.reg .b32 ta, tb, tm;\n\t"     \
            "mbarrier.test_wait.parity.shared::cta.b64 pa, [%7], %8;\n\t"                                              \
            "mbarrier.test_wait.parity.shared::cta.b64 pb, [%9], %10;\n\t"                                             \
            "setp.ne.b32 q, %5, 0;\n\t"                                                                                \
            "and.b32 tm, %6, 1;\n\tsetp.ne.b32 p0, tm, 0;\n\t"                                                        \
            "and.b32 tm, %6, 2;\n\tsetp.ne.b32 p1, tm, 0;\n\t"                                                        \
            "and.b32 tm, %6, 4;\n\tsetp.ne.b32 p2, tm, 0;\n\t"                                                        \
            "and.b32 tm, %6, 8;\n\tsetp.ne.b32 p3, tm, 0;\n\t"                                                        \
            "add.u64 a1, %2, 2;\n\tadd.u64 a2, %2, 4;\n\tadd.u64 a3, %2, 6;\n\t"                                      \
            "add.u64 b1, %3, 2;\n\tadd.u64 b2, %3, 4;\n\tadd.u64 b3, %3, 6;\n\t"                                      \
            "@p0 tcgen05.mma.cta_group::1.kind::" KIND " [%1], %2, %3, %4, q;\n\t"                                     \
            "or.pred q, q, p0;\n\t"                                                                                    \
            "@p1 tcgen05.mma.cta_group::1.kind::" KIND " [%1], a1, b1, %4, q;\n\t"                                     \
            "or.pred q, q, p1;\n\t"                                                                                    \
            "@p2 tcgen05.mma.cta_group::1.kind::" KIND " [%1], a2, b2, %4, q;\n\t"                                     \
            "or.pred q, q, p2;\n\t"                                                                                    \
            "@p3 tcgen05.mma.cta_group::1.kind::" KIND " [%1], a3, b3, %4, q;\n\t"                                     \
            "selp.u32 ta, 1, 0, pa;\n\t"                                                                               \
            "selp.u32 tb, 2, 0, pb;\n\t"                                                                               \
            "or.b32 %0, ta, tb;\n\t}"                                                                                  \
            : "=r"(res)                                                                                                \
            : "r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate), "r"(m4), "r"(barA), "r"(parA), "r"(barB), \
              "r"(parB)                                                                                                \
            : "memory");                                                                                               \
        return res;                                                                                                    \
    }
RTOSS_DEFINE_PEEK(umma_block_peek_f16, "f16")
RTOSS_DEFINE_PEEK(umma_block_peek_tf32, "tf32")
#undef RTOSS_DEFINE_PEEK
template <bool TF32>
__device__ __forceinline__ unsigned umma_block_peek(unsigned d_tmem, unsigned long long adesc, unsigned long long bdesc,
                                                    unsigned idesc, unsigned accumulate, unsigned m4, unsigned barA,
                                                    unsigned parA, unsigned barB, unsigned parB) {
    return TF32 ? umma_block_peek_tf32(d_tmem, adesc, bdesc, idesc, accumulate, m4, barA, parA, barB, parB)
                : umma_block_peek_f16(d_tmem, adesc, bdesc, idesc, accumulate, m4, barA, parA, barB, parB);
}
// Arrive on an mbarrier once all tcgen05.mma issued so far by this thread have completed.
__device__ __forceinline__ void umma_commit(unsigned bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}

__device__ __forceinline__ void tmem_ld32(unsigned taddr, unsigned (&r)[32]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
          "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]),
          "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]),
          "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr)
        : "memory");
}

template <typename T>
__device__ __forceinline__ unsigned pack2(float a, float b);
template <>
__device__ __forceinline__ unsigned pack2<__nv_bfloat16>(float a, float b) {
    __nv_bfloat162 v = __floats2bfloat162_rn(a, b);
    return *reinterpret_cast<unsigned*>(&v);
}
template <>
__device__ __forceinline__ unsigned pack2<__half>(float a, float b) {
    __half2 v = __floats2half2_rn(a, b);
    return *reinterpret_cast<unsigned*>(&v);
}

__device__ __forceinline__ void tmem_ld16(unsigned taddr, unsigned (&r)[16]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
          "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
        : "r"(taddr)
        : "memory");
}

// Sixteen consecutive filters of one position (positions as the M operand): bias, activation, rounding, packed
// two to a register in memory order.
template <typename T, int ACT>
__device__ __forceinline__ void act_pack16(const unsigned (&r)[16], const float* bias16, unsigned (&o)[8]) {
#pragma unroll
    for (int j = 0; j < 16; j += 2) {
        float v[2];
#pragma unroll
        for (int e = 0; e < 2; ++e) {
            v[e] = __uint_as_float(r[j + e]) + bias16[j + e];
            if (ACT == RTOSS_ACT_RELU) v[e] = fmaxf(v[e], 0.f);
            if (ACT == RTOSS_ACT_SILU) {
                float th;
                asm("tanh.approx.f32 %0, %1;" : "=f"(th) : "f"(0.5f * v[e]));
                v[e] = v[e] * fmaf(0.5f, th, 0.5f);
            }
        }
        o[j >> 1] = pack2<T>(v[0], v[1]);
    }
}

// Two fp32 values rounded to the 16-bit output type and packed (lo in the low half), with the ReLU folded into
// the conversion where asked for.
template <typename T, bool RELU>
__device__ __forceinline__ unsigned round_pack(float lo, float hi);
template <>
__device__ __forceinline__ unsigned round_pack<__nv_bfloat16, false>(float lo, float hi) {
    return pack2<__nv_bfloat16>(lo, hi);
}
template <>
__device__ __forceinline__ unsigned round_pack<__half, false>(float lo, float hi) {
    return pack2<__half>(lo, hi);
}
template <>
__device__ __forceinline__ unsigned round_pack<__nv_bfloat16, true>(float lo, float hi) {
    unsigned d;
    asm("cvt.rn.relu.bf16x2.f32 %0, %1, %2;" : "=r"(d) : "f"(hi), "f"(lo));
    return d;
}
template <>
__device__ __forceinline__ unsigned round_pack<__half, true>(float lo, float hi) {
    unsigned d;
    asm("cvt.rn.relu.f16x2.f32 %0, %1, %2;" : "=r"(d) : "f"(hi), "f"(lo));
    return d;
}

// SiLU of an fp32 output: v / (1 + e^-v) with the fast exponential (a few ulp: the tanh form below is good to 2^-11
// only, enough for 16-bit outputs, not for the 1e-4 bound of fp32 ones).
__device__ __forceinline__ float silu_f32(float v) { return v / (1.f + __expf(-v)); }

// Bias and activation of one accumulator value.  bs is the bias, for SiLU half the bias:
//   v * sigmoid(v) = h + h * tanh(h) with h = v / 2 = fma(acc, 0.5, b / 2): two fused multiply-adds around one
//   special-function op (tanh.approx, relative error about 2^-11: below half an ulp of bf16, about one ulp of
//   fp16).  ReLU is left to the conversion.
template <int ACT>
__device__ __forceinline__ float bias_act(unsigned acc_bits, float bs) {
    const float acc = __uint_as_float(acc_bits);
    if (ACT == RTOSS_ACT_SILU) {
        const float h = fmaf(acc, 0.5f, bs);
        float th;
        asm("tanh.approx.f32 %0, %1;" : "=f"(th) : "f"(h));
        return fmaf(h, th, h);
    }
    return acc + bs;
}

// Eight outputs of one position (four words of two 16-bit values, already rounded without activation) plus the eight
// residual values at the same place: sum in fp32, activation, one more rounding -- what a convolution without
// activation followed by an element-wise add + activation gives, bit for bit (act none and ReLU; SiLU here is the
// tanh form of the epilogue).
template <typename T, int ACT>
__device__ __forceinline__ uint4 add_residual8(uint4 o, const uint4 rv) {
    const T* oe = reinterpret_cast<const T*>(&o);
    const T* re = reinterpret_cast<const T*>(&rv);
    unsigned w[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        float v[2];
#pragma unroll
        for (int e = 0; e < 2; ++e) {
            v[e] = to_f32<T>(oe[2 * i + e]) + to_f32<T>(re[2 * i + e]);
            if (ACT == RTOSS_ACT_SILU) {
                const float h = 0.5f * v[e];
                float th;
                asm("tanh.approx.f32 %0, %1;" : "=f"(th) : "f"(h));
                v[e] = fmaf(h, th, h);
            }
        }
        w[i] = round_pack<T, ACT == RTOSS_ACT_RELU>(v[0], v[1]);
    }
    return make_uint4(w[0], w[1], w[2], w[3]);
}

// Sixteen positions of one filter (a half chunk): round, transpose through the patch, store.  See epilogue_chunks.
// With a residual operand (rbv, laid out like the output) the activation moves behind the residual add.
template <typename T, int ACT>
__device__ __forceinline__ void epilogue_half(const unsigned (&r)[16], float bs, unsigned wr, unsigned rd, unsigned tab_at,
                                              T* ybv, unsigned ry, unsigned rx, const T* rbv = nullptr, bool post = false) {
    const bool res = rbv != nullptr;   // then (unless post) bs is the plain bias and nothing is activated before the add
#pragma unroll
    for (int jp = 0; jp < kPatchRows / 2; ++jp) {
        const unsigned w = (res && !post) ? round_pack<T, false>(__uint_as_float(r[2 * jp]) + bs, __uint_as_float(r[2 * jp + 1]) + bs)
                               : round_pack<T, ACT == RTOSS_ACT_RELU>(bias_act<ACT>(r[2 * jp], bs), bias_act<ACT>(r[2 * jp + 1], bs));
        asm volatile("st.shared.u32 [%0], %1;" ::"r"(wr + jp * kPairPitch), "r"(w) : "memory");
    }
    __syncwarp();
    unsigned w[8], e[4];
    asm volatile("ld.shared.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(w[0]), "=r"(w[1]), "=r"(w[2]), "=r"(w[3]) : "r"(rd));
    asm volatile("ld.shared.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(w[4]), "=r"(w[5]), "=r"(w[6]), "=r"(w[7]) : "r"(rd + 16));
    // table entries of positions 2 jp and 2 jp + 1 (an even position: 16-byte aligned)
    asm volatile("ld.shared.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(e[0]), "=r"(e[1]), "=r"(e[2]), "=r"(e[3]) : "r"(tab_at));
    if ((e[1] >> 16) < ry && (e[1] & 0xFFFFu) < rx) {
        uint4 o = make_uint4(__byte_perm(w[0], w[1], 0x5410), __byte_perm(w[2], w[3], 0x5410), __byte_perm(w[4], w[5], 0x5410),
                             __byte_perm(w[6], w[7], 0x5410));
        if (res) {
            const uint4 rv = *reinterpret_cast<const uint4*>(rbv + e[0]);
            o = post ? add_residual8<T, RTOSS_ACT_NONE>(o, rv) : add_residual8<T, ACT>(o, rv);
        }
        *reinterpret_cast<uint4*>(ybv + e[0]) = o;
    }
    if ((e[3] >> 16) < ry && (e[3] & 0xFFFFu) < rx) {
        uint4 o = make_uint4(__byte_perm(w[0], w[1], 0x7632), __byte_perm(w[2], w[3], 0x7632), __byte_perm(w[4], w[5], 0x7632),
                             __byte_perm(w[6], w[7], 0x7632));
        if (res) {
            const uint4 rv = *reinterpret_cast<const uint4*>(rbv + e[2]);
            o = post ? add_residual8<T, RTOSS_ACT_NONE>(o, rv) : add_residual8<T, ACT>(o, rv);
        }
        *reinterpret_cast<uint4*>(ybv + e[2]) = o;
    }
    __syncwarp();
}

// One tile of the filters-as-M epilogue for one warp: its lane quarter of the accumulator stage at d_base, the
// 32-column chunks c0, c0 + c_step, ...  A warp holds 32 filters (lanes) x 16 positions (registers) at a time;
// NHWC wants the filters of one position side by side.  The shared-memory pipe (one 128-byte wavefront a cycle,
// which the tensor cores' operand reads also use) is what bounds the transpose, so it moves full wavefronts:
//   * a lane rounds two neighbouring positions of its filter into one 32-bit word and stores it to row
//     (position pair), column (filter) of the warp's patch: eight conflict-free 128-byte stores per 16 positions;
//   * lane (pair jp = lane / 4, filter group v = lane % 4) reads the eight words of its group (two 16-byte
//     loads; rows are 36 words apart, so the two rows a quarter warp touches fall on disjoint banks), splits
//     them into the low halves (position 2 jp) and the high halves (position 2 jp + 1) and writes each as one
//     16-byte store: four lanes cover the 64 contiguous bytes of a position.
// The accumulator is read sixteen columns at a time into two register sets: the load of the next sixteen is in
// flight while the current ones are processed (a load takes a few hundred cycles when all warps read at once).
// Where a position goes comes from the table built in the prologue (no division here): tab[p] = {element offset
// inside the tile, row << 16 | column}.  patch and tab are shared-memory addresses (32 bits: the accesses are
// spelled out so that none is compiled as a generic one).
template <typename T, int ACT>
__device__ __forceinline__ void epilogue_chunks(unsigned d_base, int c0, int c_step, int n_px, float bs,
                                                unsigned patch, unsigned tab, T* yb, unsigned ry, unsigned rx,
                                                int lane, const T* rb) {
    const unsigned wr = patch + lane * 4;                                       // this lane's column of the patch
    const unsigned rd = patch + (lane >> 2) * kPairPitch + (lane & 3) * 32;   // row lane / 4, filter group lane % 4
    const unsigned tab_l = tab + (unsigned)(2 * (lane >> 2)) * 8;
    T* ybv = yb + (lane & 3) * 8;
    const T* rbv = rb ? rb + (lane & 3) * 8 : nullptr;
    if (c0 >= n_px) return;
    unsigned ra[16], rb2[16];
    tmem_ld16(d_base + (unsigned)c0, ra);
    for (; c0 < n_px; c0 += c_step) {
        asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
        tmem_ld16(d_base + (unsigned)(c0 + kPatchRows), rb2);
        epilogue_half<T, ACT>(ra, bs, wr, rd, tab_l + (unsigned)c0 * 8, ybv, ry, rx, rbv);
        asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
        if (c0 + c_step < n_px) tmem_ld16(d_base + (unsigned)(c0 + c_step), ra);
        epilogue_half<T, ACT>(rb2, bs, wr, rd, tab_l + (unsigned)(c0 + kPatchRows) * 8, ybv, ry, rx, rbv);
    }
}

// The same with a residual operand.  Its values arrive by asynchronous 16-byte copies (global -> shared, no
// registers held while they fly): every lane fetches the two pieces it will add (positions 2 jp and 2 jp + 1, its
// eight filters) into its own slots of the warp's staging area, one half chunk ahead of the one being finished, so a
// load from memory has a whole half chunk of work to hide behind.  A lane reads back only what it fetched itself:
// cp.async.wait_group is all the ordering needed.  stage: shared address of the warp's kResStage bytes, two buffers
// of [2 pieces][32 lanes] x 16 bytes.
template <typename T>
__device__ __forceinline__ void fetch_residual(unsigned tab_at, const T* rbv, unsigned ry, unsigned rx, unsigned slot) {
    unsigned e[4];
    asm volatile("ld.shared.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(e[0]), "=r"(e[1]), "=r"(e[2]), "=r"(e[3]) : "r"(tab_at));
    if ((e[1] >> 16) < ry && (e[1] & 0xFFFFu) < rx)
        asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(slot), "l"(rbv + e[0]) : "memory");
    if ((e[3] >> 16) < ry && (e[3] & 0xFFFFu) < rx)
        asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(slot + 512u), "l"(rbv + e[2]) : "memory");
    asm volatile("cp.async.commit_group;" ::: "memory");
}

template <typename T, int ACT, bool POST>
__device__ __forceinline__ void epilogue_half_res(const unsigned (&r)[16], float bias, unsigned wr, unsigned rd, unsigned tab_at,
                                                  T* ybv, unsigned ry, unsigned rx, unsigned slot) {
#pragma unroll
    for (int jp = 0; jp < kPatchRows / 2; ++jp) {
        // POST: activated and rounded as without a residual (bias is then what bias_act expects); else the plain sum
        const unsigned w = POST ? round_pack<T, ACT == RTOSS_ACT_RELU>(bias_act<ACT>(r[2 * jp], bias), bias_act<ACT>(r[2 * jp + 1], bias))
                                : round_pack<T, false>(__uint_as_float(r[2 * jp]) + bias, __uint_as_float(r[2 * jp + 1]) + bias);
        asm volatile("st.shared.u32 [%0], %1;" ::"r"(wr + jp * kPairPitch), "r"(w) : "memory");
    }
    __syncwarp();
    unsigned w[8], e[4];
    asm volatile("ld.shared.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(w[0]), "=r"(w[1]), "=r"(w[2]), "=r"(w[3]) : "r"(rd));
    asm volatile("ld.shared.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(w[4]), "=r"(w[5]), "=r"(w[6]), "=r"(w[7]) : "r"(rd + 16));
    asm volatile("ld.shared.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(e[0]), "=r"(e[1]), "=r"(e[2]), "=r"(e[3]) : "r"(tab_at));
    if ((e[1] >> 16) < ry && (e[1] & 0xFFFFu) < rx) {
        uint4 rv;
        asm volatile("ld.shared.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(rv.x), "=r"(rv.y), "=r"(rv.z), "=r"(rv.w) : "r"(slot));
        const uint4 o = make_uint4(__byte_perm(w[0], w[1], 0x5410), __byte_perm(w[2], w[3], 0x5410),
                                   __byte_perm(w[4], w[5], 0x5410), __byte_perm(w[6], w[7], 0x5410));
        *reinterpret_cast<uint4*>(ybv + e[0]) = add_residual8<T, POST ? RTOSS_ACT_NONE : ACT>(o, rv);
    }
    if ((e[3] >> 16) < ry && (e[3] & 0xFFFFu) < rx) {
        uint4 rv;
        asm volatile("ld.shared.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(rv.x), "=r"(rv.y), "=r"(rv.z), "=r"(rv.w) : "r"(slot + 512u));
        const uint4 o = make_uint4(__byte_perm(w[0], w[1], 0x7632), __byte_perm(w[2], w[3], 0x7632),
                                   __byte_perm(w[4], w[5], 0x7632), __byte_perm(w[6], w[7], 0x7632));
        *reinterpret_cast<uint4*>(ybv + e[2]) = add_residual8<T, POST ? RTOSS_ACT_NONE : ACT>(o, rv);
    }
    __syncwarp();
}

template <typename T, int ACT, bool POST>
__device__ __forceinline__ void epilogue_chunks_res(unsigned d_base, int c0, int c_step, int n_px, float bias,
                                                    unsigned patch, unsigned tab, T* yb, unsigned ry, unsigned rx,
                                                    int lane, const T* rb, unsigned stage) {
    const unsigned wr = patch + lane * 4;
    const unsigned rd = patch + (lane >> 2) * kPairPitch + (lane & 3) * 32;
    const unsigned tab_l = tab + (unsigned)(2 * (lane >> 2)) * 8;
    T* ybv = yb + (lane & 3) * 8;
    const T* rbv = rb + (lane & 3) * 8;
    if (c0 >= n_px) return;
    const unsigned slot0 = stage + (unsigned)lane * 16, slot1 = slot0 + 1024u;
    unsigned ra[16], rb2[16];
    fetch_residual<T>(tab_l + (unsigned)c0 * 8, rbv, ry, rx, slot0);
    tmem_ld16(d_base + (unsigned)c0, ra);
    for (; c0 < n_px; c0 += c_step) {
        fetch_residual<T>(tab_l + (unsigned)(c0 + kPatchRows) * 8, rbv, ry, rx, slot1);
        asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
        tmem_ld16(d_base + (unsigned)(c0 + kPatchRows), rb2);
        asm volatile("cp.async.wait_group 1;" ::: "memory");   // the pieces of this half are in
        epilogue_half_res<T, ACT, POST>(ra, bias, wr, rd, tab_l + (unsigned)c0 * 8, ybv, ry, rx, slot0);
        const bool more = c0 + c_step < n_px;
        if (more)
            fetch_residual<T>(tab_l + (unsigned)(c0 + c_step) * 8, rbv, ry, rx, slot0);
        else
            asm volatile("cp.async.commit_group;" ::: "memory");   // keeps the group count in step
        asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
        if (more) tmem_ld16(d_base + (unsigned)(c0 + c_step), ra);
        asm volatile("cp.async.wait_group 1;" ::: "memory");
        epilogue_half_res<T, ACT, POST>(rb2, bias, wr, rd, tab_l + (unsigned)(c0 + kPatchRows) * 8, ybv, ry, rx, slot1);
    }
    asm volatile("cp.async.wait_group 0;" ::: "memory");
}

// Split K, second half.  Every CTA of the cluster owns the 32-column chunks c of the tile with c % KS == its rank
// (its local chunk lc = c / KS) and holds, in its own shared memory at `buf`, what each of the KS shares summed
// for them: share i, local chunk lc, column col, accumulator lane row at ((i * n_lc + lc) * 32 + col) * 128 + row
// floats.  The owned chunks are finished as half chunks of 16 columns dealt to the four warps of a lane quarter.
template <typename T, int ACT>
__device__ __forceinline__ void epilogue_from_shares(unsigned buf, int KS, int rank, int n_lc, int sub, int row, int n_px, float bs,
                                                     bool vec_ok, bool co_ok, unsigned patch, unsigned tab, const uint2* pos_tab,
                                                     T* yb, unsigned ry, unsigned rx, int lane, const T* rb, bool post) {
    const unsigned wr = patch + lane * 4;
    const unsigned rd = patch + (lane >> 2) * kPairPitch + (lane & 3) * 32;
    const unsigned tab_l = tab + (unsigned)(2 * (lane >> 2)) * 8;
    T* ybv = yb + (lane & 3) * 8;
    const T* rbv = rb ? rb + (lane & 3) * 8 : nullptr;
    for (int t = sub; t < 2 * n_lc; t += 4) {
        const int lc = t >> 1, c0 = (lc * KS + rank) * 32 + (t & 1) * kPatchRows;   // first column of the half chunk
        if (c0 >= n_px) continue;
        float sum[kPatchRows];
#pragma unroll
        for (int j = 0; j < kPatchRows; ++j) sum[j] = 0.f;
        for (int i = 0; i < KS; ++i) {
            const unsigned q = buf + (unsigned)((((i * n_lc + lc) * 32 + (t & 1) * kPatchRows) * 128 + row) * 4);
#pragma unroll
            for (int j = 0; j < kPatchRows; ++j) {
                float v;
                asm volatile("ld.shared.f32 %0, [%1];" : "=f"(v) : "r"(q + j * 512));
                sum[j] += v;
            }
        }
        unsigned r[16];
#pragma unroll
        for (int j = 0; j < kPatchRows; ++j) r[j] = __float_as_uint(sum[j]);
        bool done = false;
        if constexpr (sizeof(T) == 2) {
            if (vec_ok) {
                epilogue_half<T, ACT>(r, bs, wr, rd, tab_l + (unsigned)c0 * 8, ybv, ry, rx, rbv, post);
                done = true;
            }
        }
        if (!done) {
            constexpr bool f32 = sizeof(T) == 4;   // (fp32: bs is the plain bias and SiLU the exponential form)
#pragma unroll
            for (int j = 0; j < kPatchRows; ++j) {
                const uint2 e = pos_tab[c0 + j];
                if (co_ok && (e.y >> 16) < ry && (e.y & 0xFFFFu) < rx) {
                    float v;
                    if (rb && post) {   // activate, round, add the residual, round
                        v = f32 ? (ACT == RTOSS_ACT_SILU ? silu_f32(__uint_as_float(r[j]) + bs) : __uint_as_float(r[j]) + bs) : bias_act<ACT>(r[j], bs);
                        if (ACT == RTOSS_ACT_RELU) v = fmaxf(v, 0.f);
                        v = to_f32<T>(from_f32<T>(v)) + to_f32<T>(rb[e.x + lane]);
                    } else if (rb) {   // round, add the residual, activate, round
                        v = to_f32<T>(from_f32<T>(__uint_as_float(r[j]) + bs)) + to_f32<T>(rb[e.x + lane]);
                        if (ACT == RTOSS_ACT_RELU) v = fmaxf(v, 0.f);
                        if (ACT == RTOSS_ACT_SILU) {
                            if (f32) {
                                v = silu_f32(v);
                            } else {
                                float th;
                                asm("tanh.approx.f32 %0, %1;" : "=f"(th) : "f"(0.5f * v));
                                v = fmaf(0.5f * v, th, 0.5f * v);
                            }
                        }
                    } else {
                        v = f32 ? (ACT == RTOSS_ACT_SILU ? silu_f32(__uint_as_float(r[j]) + bs) : __uint_as_float(r[j]) + bs) : bias_act<ACT>(r[j], bs);
                        if (ACT == RTOSS_ACT_RELU) v = fmaxf(v, 0.f);
                    }
                    yb[e.x + lane] = from_f32<T>(v);
                }
            }
        }
    }
}

// Which problem a unit of the launch's list belongs to, and its index inside that problem.  A CTA's units ascend, so
// the search goes on from the problem of its previous unit (`from`).
template <bool kMulti, typename G>
__device__ __forceinline__ int find_problem(const G& g, int unit, int& local, int from = 0) {
    if (!kMulti) {   // a launch of one problem: the index is a compile-time constant
        local = unit;
        return 0;
    }
    int pi = from;
    while (pi + 1 < g.n_prob && unit >= g.unit_end[pi]) ++pi;
    local = unit - (pi ? g.unit_end[pi - 1] : 0);
    return pi;
}

// n / d for n < 2^31 by a multiplication: md = {ceil(2^(31 + l) / d), l - 1} with l = ceil(log2 d), or {0, 0} for d = 1
// (exact: the multiplier's error, below 2^l / d <= 2 parts in 2^(31 + l), cannot carry a quotient of n < 2^31 over).
__host__ __device__ __forceinline__ void magic_of(int d, unsigned (&md)[2]) {
    md[0] = md[1] = 0;
    if (d <= 1) return;
    int l = 0;
    while ((1ll << l) < d) ++l;
    md[0] = (unsigned)((((unsigned long long)1 << (31 + l)) + (unsigned)d - 1) / (unsigned)d);
    md[1] = (unsigned)(l - 1);
}
__device__ __forceinline__ int fdiv(int n, const unsigned (&md)[2]) {
    return md[0] ? (int)(__umulhi((unsigned)n, md[0]) >> md[1]) : n;
}
// A unit of problem a taken apart.
struct TileIdx {
    int ks, cot, tx, ty, n;
};
__device__ __forceinline__ TileIdx tile_of(const TcArgs& a, int local) {
    TileIdx t;
    int rest = fdiv(local, a.div_ks);
    t.ks = local - rest * a.KS;
    int q = fdiv(rest, a.div_co);
    t.cot = rest - q * a.co_tiles;
    rest = q;
    q = fdiv(rest, a.div_tx);
    t.tx = rest - q * a.tiles_x;
    rest = q;
    t.n = fdiv(rest, a.div_ty);
    t.ty = rest - t.n * a.tiles_y;
    return t;
}

// A ring of stages with one "full" and one "empty" mbarrier per stage: position s and, per stage, the parity of the
// phase its next use belongs to (bit i of par = stage i).  The parities are kept per stage because the problems of a
// launch may run with different ring depths: the stages then do not all have the same number of uses behind them.
struct Ring {
    int s = 0;
    unsigned par = 0;
    __device__ __forceinline__ unsigned parity() const { return (par >> s) & 1u; }
    __device__ __forceinline__ void advance(int n) {
        par ^= 1u << s;
        if (++s == n) s = 0;
    }
};

// Dependent problems of one launch: waits (bounded) until every problem named in dep_mask has all its outputs written,
// then orders this thread's coming bulk copies behind what it has seen.  The writers' side is at the end of the
// epilogue's tile loop.
template <typename G>
__device__ __forceinline__ bool wait_deps(const G& g, unsigned dep_mask) {
    const long long t0 = clock64();
    while (dep_mask) {
        const int j = __ffs((int)dep_mask) - 1;
        dep_mask &= dep_mask - 1;
        const unsigned target = g.prob[j].done_target;
        for (;;) {
            unsigned seen;
            asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(seen) : "l"(g.done + j) : "memory");
            if (seen >= target) break;
            if (clock64() - t0 > g.wait_cycles) return false;
            __nanosleep(100);
        }
    }
    // the outputs were written with ordinary stores; the copies that fetch them go through the asynchronous proxy
    asm volatile("fence.proxy.async;" ::: "memory");
    return true;
}

template <typename T, typename G>
__global__ void __launch_bounds__(kTcThreads, 1)
conv_tc_kernel(const __grid_constant__ G g) {
    constexpr bool kMulti = sizeof(G) > sizeof(TcLaunch1);
    constexpr bool kF32 = sizeof(T) == 4;   // fp32 data: tf32 instructions, three products per tap (see the head of the file)
    extern __shared__ unsigned char smem_dyn[];
    // tiles need 1024-byte alignment for the 128-byte swizzle pattern
    const unsigned base = (smem_u32(smem_dyn) + 1023u) & ~1023u;
    const unsigned sA = base;                                        // the ring area: a problem's [NA][a_stage], then its [NB][b_stage]
    const unsigned sBar = sA + (unsigned)g.ring_bytes;               // barriers, 8 bytes each
    const unsigned bar_fullA = sBar, bar_emptyA = sBar + 8 * kMaxA;
    const unsigned bar_fullB = bar_emptyA + 8 * kMaxA, bar_emptyB = bar_fullB + 8 * kMaxB;
    const unsigned bar_accFull = bar_emptyB + 8 * kMaxB, bar_accEmpty = bar_accFull + 16;
    const unsigned bar_loFull = bar_accEmpty + 16;   // fp32: activation stage split into heads and remainders
    // A CTA passing from a problem to one of another ring geometry: the MMA thread commits here once everything it
    // issued for the old problem has completed, i.e. has read its operands; both producers wait for that before they
    // write the first stage of the new layout over the old one.
    const unsigned bar_switch = bar_loFull + 8 * kMaxA;
    const unsigned s_tmem_ptr = bar_switch + 16;   // (what follows needs 16-byte alignment)
    volatile unsigned* tmem_ptr_gen = reinterpret_cast<volatile unsigned*>(smem_dyn + (s_tmem_ptr - smem_u32(smem_dyn)));
    unsigned char* epi_patch = smem_dyn + (s_tmem_ptr + 16 - smem_u32(smem_dyn));  // [kEpiWarps][kPatchBytes], 16-byte aligned
    uint2* pos_tab_all = reinterpret_cast<uint2*>(epi_patch + kEpiWarps * kPatchBytes);  // [n_tabs][kMaxPx]
    const unsigned s_tab_all = s_tmem_ptr + 16 + kEpiWarps * kPatchBytes;                // the same, as a shared address
    const unsigned s_res = sA + (unsigned)g.res_off;   // [kEpiWarps][kResStage], present when a call has a residual operand

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int n_tiles = g.unit_end[g.n_prob - 1];  // units of work over all problems: (tile, share of the channel blocks)
    // Programmatic dependent launch: the next kernel of the stream may start its own prologue now (on SMs this
    // grid leaves free); it reads or writes nothing before its own griddepcontrol.wait.
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");

    if (threadIdx.x == 0) {
        for (int i = 0; i < g.max_na; ++i) {
            mbar_init(bar_fullA + 8 * i, 1);
            mbar_init(bar_emptyA + 8 * i, 1);
            mbar_init(bar_loFull + 8 * i, 1);
        }
        for (int i = 0; i < g.max_nb; ++i) {
            mbar_init(bar_fullB + 8 * i, 1);
            mbar_init(bar_emptyB + 8 * i, 1);
        }
        mbar_init(bar_switch, 1);
        for (int i = 0; i < g.AS; ++i) {
            mbar_init(bar_accFull + 8 * i, 1);
            mbar_init(bar_accEmpty + 8 * i, kEpiWarps);
        }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        for (int i = 0; i < g.n_prob; ++i) {
            asm volatile("prefetch.tensormap [%0];" ::"l"(&g.tmA[i]) : "memory");
            asm volatile("prefetch.tensormap [%0];" ::"l"(&g.tmB[i]) : "memory");
        }
    }
    // Where position p of a tile's list lies: the same for every tile (the tile's origin and the image's edges
    // come in per tile), so the epilogue looks it up instead of dividing.  {element offset from the tile's first
    // output, row << 16 | column}; positions that are no output (pitch padding, the list's tail) get 0xFFFFFFFF.
    for (int q = threadIdx.x; q < g.n_tabs * kMaxPx; q += kTcThreads) {
        int owner = 0;   // (any problem that uses the table describes it)
        while (owner + 1 < g.n_prob && g.prob[owner].tab != q / kMaxPx) ++owner;
        const TcArgs& a = g.prob[owner];
        const int p = q % kMaxPx;
        const int oyl = p / a.Wq, oxl = p - oyl * a.Wq;
        const bool is_out = p < a.N_px && oyl < a.TH && oxl < a.TW;
        pos_tab_all[q] = make_uint2((unsigned)((oyl * a.Wo + oxl) * a.y_c_stride), is_out ? (unsigned)(oyl << 16 | oxl) : 0xFFFFFFFFu);
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(s_tmem_ptr), "r"(g.tmem_cols)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const unsigned tmem_base = *tmem_ptr_gen;
    // Everything above (barriers, TMEM, descriptor prefetch) touched no tensor.  What depends on the kernels before this
    // one in the stream -- the activations, the bias, the residual operand, and y, which they may still read -- is only
    // touched behind a griddepcontrol.wait, which the activation producer and the epilogue warps execute at the top of
    // their roles.  The weights and the issue words are not: they are constant while a network runs, and the kernels
    // that write them (packing) never let a successor start early, so the weight producer and the MMA thread begin at
    // once and the weight ring is full by the time the activations may be fetched.

    // Every role walks the same list of tiles: tile = blockIdx.x, + gridDim.x, ...  A tile is (image,
    // row band, filter tile) with the filter tile fastest, so CTAs working side by side read the same
    // activations from L2.  Stage counters run on across tiles, which lets the producer fetch the next
    // tile's operands while the current one is still being multiplied, and the two accumulator stages
    // let the epilogue of one tile run under the MMAs of the next.
    if (warp == 0) {
        // ---------------- TMA producer of the activations.  Issuing a bulk copy keeps its thread busy for some
        // hundred cycles whatever the size, so the activations and the weights have a producer thread each, and a
        // weight stage (G taps) is ONE copy.
        asm volatile("griddepcontrol.wait;" ::: "memory");   // the activations come from the kernels before this one
        if (kF32 || lane == 0) {
            // (fp32: all 32 lanes walk the loop; lane 0 issues the copies, then the warp splits the block that arrived)
            bool ok = true;
            Ring ra;
            int pi = 0, cur_pi = -1;
            unsigned n_sw = 0;   // geometry changes so far
            for (int unit = blockIdx.x; unit < n_tiles && ok; unit += gridDim.x) {
                int local;
                pi = find_problem<kMulti>(g, unit, local, pi);
                const TcArgs& a = g.prob[pi];
                if (kMulti && pi != cur_pi) {
                    // another problem: if its rings are laid out differently, the old ones must have run empty; if it
                    // depends on problems of this launch, they must be complete
                    const bool regeo = cur_pi >= 0 && a.geo != g.prob[cur_pi].geo;
                    if (lane == 0) {
                        if (regeo) ok = mbar_wait(bar_switch, n_sw & 1u, g.wait_cycles);
                        if (ok && a.dep_mask) ok = wait_deps(g, a.dep_mask);
                    }
                    if (regeo) {
                        ++n_sw;
                        ra.s = 0;
                    }
                    cur_pi = pi;
                }
                const TileIdx ti = tile_of(a, local);
                const int ks = ti.ks, n = ti.n;
                const int y0 = ti.ty * a.TH, x0 = ti.tx * a.TW;
                const int cb_end = min(a.ncb, (ks + 1) * a.cb_per);
                for (int cb = ks * a.cb_per; cb < cb_end; ++cb) {
                    const int sa = ra.s;
                    const unsigned pa = ra.parity();
                    if (lane == 0) {
                        ok = ok && mbar_wait(bar_emptyA + 8 * sa, pa ^ 1, g.wait_cycles);
                        if (ok) {
                            mbar_expect_tx(bar_fullA + 8 * sa, a.a_tx_bytes * a.n_sub);
                            for (int sub = 0; sub < a.n_sub; ++sub)
                                tma_load_4d(sA + sa * a.a_stage + sub * a.sub_bytes, &g.tmA[pi], cb * a.cb_ch, x0 * a.S + a.x_add[sub],
                                            y0 * a.S + a.y_add[sub], n, bar_fullA + 8 * sa);
                        }
                    }
                    if (kF32) {
                        // Split the block: x = head + remainder, head = the 19 leading bits (what a tf32 operand holds), in
                        // place; the remainder (exact in fp32) goes to the second half of the stage.  Plain loads and stores
                        // of this warp; the fence hands them to the proxy the tensor core reads through; then the stage is
                        // announced to the MMA thread.  Any word may be split: rows the copy did not write are never outputs.
                        ok = __shfl_sync(0xFFFFFFFFu, (int)ok, 0) != 0;
                        if (ok) {
                            if (lane == 0) ok = mbar_wait(bar_fullA + 8 * sa, pa, g.wait_cycles);
                            ok = __shfl_sync(0xFFFFFFFFu, (int)ok, 0) != 0;
                        }
                        if (ok) {
                            const unsigned src = sA + sa * a.a_stage, dst = src + (unsigned)a.lo_off;
                            const int n16 = (a.n_sub * a.sub_bytes) >> 4;
#pragma unroll 4
                            for (int i = lane; i < n16; i += 32) {
                                unsigned v[4], h[4], l[4];
                                asm volatile("ld.shared.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]) : "r"(src + 16u * i));
#pragma unroll
                                for (int e = 0; e < 4; ++e) {
                                    h[e] = v[e] & 0xFFFFE000u;
                                    l[e] = __float_as_uint(__fsub_rn(__uint_as_float(v[e]), __uint_as_float(h[e])));
                                }
                                asm volatile("st.shared.v4.u32 [%0], {%1, %2, %3, %4};" ::"r"(src + 16u * i), "r"(h[0]), "r"(h[1]), "r"(h[2]), "r"(h[3]) : "memory");
                                asm volatile("st.shared.v4.u32 [%0], {%1, %2, %3, %4};" ::"r"(dst + 16u * i), "r"(l[0]), "r"(l[1]), "r"(l[2]), "r"(l[3]) : "memory");
                            }
                            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                            __syncwarp();
                            if (lane == 0) asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar_loFull + 8 * sa) : "memory");
                        }
                    }
                    if (!ok) break;
                    ra.advance(a.NA);
                }
            }
            if (!ok && lane == 0) atomicExch(g.status, 1);
        }
        __syncwarp();  // lanes 1..31 wait here for lane 0: the warp reaches the final barrier as one
    } else if (warp == kWeightWarp) {
        // ---------------- TMA producer of the weights: per tile and channel block, taps / G stages of G taps each
        if (lane == 0) {
            bool ok = true;
            Ring rb;
            int pi = 0, cur_pi = -1;
            unsigned n_sw = 0;
            for (int unit = blockIdx.x; unit < n_tiles && ok; unit += gridDim.x) {
                int local;
                pi = find_problem<kMulti>(g, unit, local, pi);
                const TcArgs& a = g.prob[pi];
                if (kMulti && pi != cur_pi) {
                    if (cur_pi >= 0 && a.geo != g.prob[cur_pi].geo) {   // the old rings must have run empty
                        ok = mbar_wait(bar_switch, n_sw & 1u, g.wait_cycles);
                        if (!ok) break;
                        ++n_sw;
                        rb.s = 0;
                    }
                    cur_pi = pi;
                }
                const unsigned sB = sA + a.sB_off;
                const TileIdx ti = tile_of(a, local);
                const int ks = ti.ks, cot = ti.cot;
                const int co0 = cot * (a.pxm ? a.n_cols : kMTile);
                const int cb_end = min(a.ncb, (ks + 1) * a.cb_per);
                for (int cb = ks * a.cb_per; cb < cb_end && ok; ++cb) {
                    for (int t0 = 0; t0 < a.taps; t0 += a.G) {
                        const int sb = rb.s;
                        ok = mbar_wait(bar_emptyB + 8 * sb, rb.parity() ^ 1u, g.wait_cycles);
                        if (!ok) break;
                        // (failure-detection hook: the launch's very first weight copy is withheld, so the wait for it runs out)
                        if (!(g.inject == 1 && unit == (int)blockIdx.x && cb == ks * a.cb_per && t0 == 0)) {
                            mbar_expect_tx(bar_fullB + 8 * sb, a.b_tx_bytes * a.G);
                            tma_load_3d(sB + sb * a.b_stage, &g.tmB[pi], cb * a.cb_ch, co0, t0, bar_fullB + 8 * sb);
                        }
                        rb.advance(a.NB);
                    }
                }
            }
            if (!ok) atomicExch(g.status, 4);
        }
        __syncwarp();
    } else if (warp == 1) {
        // ---------------- MMA issuer
        if (lane == 0) {
            // One thread issues every tcgen05.mma, so the instructions between two of them are the budget: with one or
            // two instructions per tap (few channels, or few filters with the positions as M) the tensor pipe waits
            // for this thread.  Hence: ring positions and phases are carried as counters (no division), a descriptor
            // is a constant high word plus address / 16 in the low word (addresses stay below 2^18: adding never
            // carries out of the field), a tap's offset is a register picked by a compile-time index (the taps of
            // a 3x3 layer are unrolled), and K steps (+2 = 32 bytes = 16 channels) or the second half of the
            // positions (+1024 = 128 rows) are additions.
            bool ok = true;
            const unsigned desc_lo0 = (unsigned)make_sw_desc(0, 128);   // (the lower word does not depend on the row size)
            // per problem (recomputed when a tile belongs to another problem than the one before)
            unsigned tap16[9], wtile16 = 0, idesc = 0, hi_cols = 0, astage16 = 0, bstage16 = 0, sB = 0, desc_hi = 0, half16 = 0;
            int NA = 1, NB = 1;
            bool pxm = false, two = false, unrolled9 = false;
            int cur_pi = -1, pi = 0;
            const unsigned bar_rdyA = kF32 ? bar_loFull : bar_fullA;   // the barrier that says an activation stage may be read
            Ring ra, rb;
            int as = 0, n_done = 0;
            unsigned pacc = 0;                  // phase parity of the accumulator ring
            unsigned peek = 0;                  // what umma_block_peek saw of the stages now current
            int since_res = 1 << 20;            // tiles issued since this CTA's last tile with a residual operand
            auto mk = [&desc_hi](unsigned lo) { return ((unsigned long long)desc_hi << 32) | lo; };
            // all instructions of one tap: the K slabs named by m4 (times two halves of positions with the positions as M)
            auto issue_tap = [&](unsigned d_base, unsigned wl, unsigned xl, unsigned m4, unsigned& acc) {
                if (pxm) {
#pragma unroll
                    for (int k4 = 0; k4 < kKBlock / 16; ++k4) {
                        if (m4 & (1u << k4)) {
                            umma_f16<kF32>(d_base, mk(xl + 2 * k4), mk(wl + 2 * k4), idesc, acc);
                            if (two) umma_f16<kF32>(d_base + hi_cols, mk(xl + half16 + 2 * k4), mk(wl + 2 * k4), idesc, acc);
                            acc = 1;
                        }
                    }
                } else {
#pragma unroll
                    for (int k4 = 0; k4 < kKBlock / 16; ++k4) {
                        if (m4 & (1u << k4)) {
                            umma_f16<kF32>(d_base, mk(wl + 2 * k4), mk(xl + 2 * k4), idesc, acc);
                            acc = 1;
                        }
                    }
                }
            };
            for (int tile = blockIdx.x; tile < n_tiles && ok; tile += gridDim.x, ++n_done) {
                int local;
                pi = find_problem<kMulti>(g, tile, local, pi);
                const TcArgs& a = g.prob[pi];
                if (pi != cur_pi) {
                    if (kMulti && cur_pi >= 0 && a.geo != g.prob[cur_pi].geo) {
                        if (a.over_res) {
                            // The new rings cover the staging area of residual operands.  An epilogue that may still use it
                            // belongs to one of this CTA's last AS tiles (the accumulator stage of an older one has been
                            // waited for since), and only if that tile had a residual operand: `since_res` tiles ago or earlier.
                            int as_b = as;
                            unsigned pacc_b = pacc;
                            for (int i = 0; i < g.AS && i < n_done && ok; ++i) {
                                if (--as_b < 0) {
                                    as_b = g.AS - 1;
                                    pacc_b ^= 1;
                                }
                                if (i >= since_res) ok = mbar_wait(bar_accEmpty + 8 * as_b, pacc_b, g.wait_cycles);
                            }
                            if (!ok) break;
                        }
                        // rings of another layout: the producers may write them once everything issued so far has read its operands
                        umma_commit(bar_switch);
                        ra.s = rb.s = 0;
                        peek = 0;
                    }
                    cur_pi = pi;
                    astage16 = a.a_stage >> 4;
                    bstage16 = a.b_stage >> 4;
                    sB = sA + a.sB_off;
                    NA = a.NA;
                    NB = a.NB;
#pragma unroll
                    for (int t = 0; t < 9; ++t) tap16[t] = (unsigned)(a.tap_sub[t] * a.sub_bytes + a.tap_shift[t] * a.row_bytes) >> 4;
                    wtile16 = (unsigned)(a.w_rows * a.row_bytes) >> 4;
                    desc_hi = a.desc_hi;
                    half16 = (unsigned)(128 * a.row_bytes) >> 4;   // the second 128 positions of a tile
                    idesc = a.idesc;
                    hi_cols = (unsigned)a.n_cols;
                    pxm = a.pxm != 0;
                    two = a.MH == 2;
                    unrolled9 = !kF32 && a.taps == 9 && a.G == 3;
                }
                const TileIdx ti = tile_of(a, local);
                const int ks = ti.ks, cb_end = min(a.ncb, (ks + 1) * a.cb_per);
                // which (tap, slab) pairs of this filter tile hold kept weights: one word per channel block, the next
                // block's word asked for while this block's instructions go out
                const unsigned long long* iss = a.issue ? a.issue + (size_t)ti.cot * a.ncb : nullptr;
                unsigned long long bits = iss ? __ldg(iss + ks * a.cb_per) : ~0ull;
                ok = mbar_wait(bar_accEmpty + 8 * as, pacc ^ 1, g.wait_cycles);  // epilogue has drained this stage
                if (!ok) break;
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                const unsigned d_base = tmem_base + (unsigned)(as * g.acc_stride);
                unsigned acc = 0;  // the first instruction of a tile overwrites the accumulator
                int left = a.Cin - ks * a.cb_per * a.cb_ch;
                for (int cb = ks * a.cb_per; cb < cb_end && ok; ++cb, left -= a.cb_ch) {
                    // 32-byte slabs of this block that hold channels (the rest of the row is TMA zero fill)
                    const int nk4 = (min(left, a.cb_ch) + a.slab_ch - 1) / a.slab_ch;
                    const unsigned nkmask = (1u << nk4) - 1u;
                    const int sa = ra.s;
                    if (a.taps == 1) {
                        const int sb = rb.s;
                        if (!(peek & 1u)) ok = mbar_wait(bar_rdyA + 8 * sa, ra.parity(), g.wait_cycles);
                        if (ok && !(peek & 2u)) ok = mbar_wait(bar_fullB + 8 * sb, rb.parity(), g.wait_cycles);
                        if (!ok) break;
                        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                        ra.advance(NA);   // now at the next stages, which the instruction below looks at
                        rb.advance(NB);
                        const int sa_n = ra.s, sb_n = rb.s;
                        const unsigned pa_n = ra.parity(), pb_n = rb.parity();
                        const unsigned wl0 = desc_lo0 + (sB >> 4) + (unsigned)sb * bstage16;
                        const unsigned xl0 = desc_lo0 + (sA >> 4) + (unsigned)sa * astage16;
                        if (!pxm) {
                            peek = umma_block_peek<kF32>(d_base, mk(wl0), mk(xl0), idesc, acc, nkmask, bar_rdyA + 8 * sa_n, pa_n,
                                                   bar_fullB + 8 * sb_n, pb_n);
                        } else {
                            // positions on M: the first 128 positions with the look ahead, then the second 128
                            peek = umma_block_peek<kF32>(d_base, mk(xl0), mk(wl0), idesc, acc, nkmask, bar_rdyA + 8 * sa_n, pa_n,
                                                   bar_fullB + 8 * sb_n, pb_n);
                            if (two) {
                                unsigned acc2 = acc;
#pragma unroll
                                for (int k4 = 0; k4 < kKBlock / 16; ++k4) {
                                    if (k4 < nk4) {
                                        umma_f16<kF32>(d_base + hi_cols, mk(xl0 + half16 + 2 * k4), mk(wl0 + 2 * k4), idesc, acc2);
                                        acc2 = 1;
                                    }
                                }
                            }
                        }
                        acc = 1;
                        umma_commit(bar_emptyB + 8 * sb);
                        umma_commit(bar_emptyA + 8 * sa);
                        continue;
                    }
                    const unsigned long long bits_n = (iss && cb + 1 < cb_end) ? __ldg(iss + cb + 1) : ~0ull;
                    if (!(peek & 1u)) ok = mbar_wait(bar_rdyA + 8 * sa, ra.parity(), g.wait_cycles);   // (peek stays 0 on the paths that do not look ahead)
                    if (!ok) break;
                    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                    const unsigned xl0 = desc_lo0 + (sA >> 4) + (unsigned)sa * astage16;
                    ra.advance(NA);   // (sa stays this block's stage; ra is at the next one, which the look ahead reads)
                    if (unrolled9) {
                        const int sa_n = ra.s;
                        const unsigned pa_n = ra.parity();
#pragma unroll
                        for (int s3 = 0; s3 < 3; ++s3) {
                            const int sb = rb.s;
                            if (!(peek & 2u)) ok = ok && mbar_wait(bar_fullB + 8 * sb, rb.parity(), g.wait_cycles);
                            if (ok) {
                                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                                const unsigned wl0 = desc_lo0 + (sB >> 4) + (unsigned)sb * bstage16;
                                const unsigned m_first = (unsigned)(bits >> (12 * s3)) & nkmask;
                                rb.advance(NB);
                                if (!pxm) {
                                    // the first tap of the stage goes out together with a look at the next stages
                                    peek = umma_block_peek<kF32>(d_base, mk(wl0), mk(xl0 + tap16[s3 * 3]), idesc, acc, m_first,
                                                           bar_rdyA + 8 * sa_n, pa_n, bar_fullB + 8 * rb.s, rb.parity());
                                    if (m_first) acc = 1;
#pragma unroll
                                    for (int i = 1; i < 3; ++i)
                                        issue_tap(d_base, wl0 + i * wtile16, xl0 + tap16[s3 * 3 + i],
                                                  (unsigned)(bits >> (12 * s3 + 4 * i)) & nkmask, acc);
                                } else {
#pragma unroll
                                    for (int i = 0; i < 3; ++i)
                                        issue_tap(d_base, wl0 + i * wtile16, xl0 + tap16[s3 * 3 + i],
                                                  (unsigned)(bits >> (12 * s3 + 4 * i)) & nkmask, acc);
                                }
                                umma_commit(bar_emptyB + 8 * sb);  // this weight stage may be refilled once the MMAs have read it
                            }
                        }
                    } else {
                        for (int t0 = 0; t0 < a.taps && ok; t0 += a.G) {
                            const int sb = rb.s;
                            ok = mbar_wait(bar_fullB + 8 * sb, rb.parity(), g.wait_cycles);
                            if (!ok) break;
                            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                            const unsigned wl0 = desc_lo0 + (sB >> 4) + (unsigned)sb * bstage16;
                            for (int i = 0; i < a.G; ++i) {
                                // weight tile v of the block: tap v (16-bit data); fp32: the heads of tap v, then (v >= 9
                                // resp. 1) the remainders of tap v - 9.  Heads meet the activations' heads and remainders,
                                // remainders the heads only.
                                const int v = t0 + i, t = v >= a.taps_real ? v - a.taps_real : v;
                                const unsigned off = (unsigned)(a.tap_sub[t] * a.sub_bytes + a.tap_shift[t] * a.row_bytes) >> 4;
                                const unsigned m4 = (unsigned)(bits >> (4 * t)) & nkmask;
                                issue_tap(d_base, wl0 + i * wtile16, xl0 + off, m4, acc);
                                if (kF32 && v < a.taps_real) issue_tap(d_base, wl0 + i * wtile16, xl0 + off + ((unsigned)a.lo_off >> 4), m4, acc);
                            }
                            umma_commit(bar_emptyB + 8 * sb);
                            rb.advance(NB);
                        }
                    }
                    if (ok) umma_commit(bar_emptyA + 8 * sa);
                    bits = bits_n;
                }
                if (ok) umma_commit(bar_accFull + 8 * as);
                since_res = a.resid ? 0 : since_res + 1;
                if (++as == g.AS) {
                    as = 0;
                    pacc ^= 1;
                }
            }
            // TMEM may only be released after the epilogue has drained the last tiles: the last min(AS, tiles done)
            // stages used, walking backwards from the ring position
            for (int i = 0; i < g.AS && i < n_done && ok && g.prob[0].KS == 1; ++i) {   // (split K: the cluster barriers below order it)
                if (--as < 0) {
                    as = g.AS - 1;
                    pacc ^= 1;
                }
                ok = mbar_wait(bar_accEmpty + 8 * as, pacc, g.wait_cycles);
            }
            if (!ok) atomicExch(g.status, 2);
        }
        __syncwarp();
    } else {
        // ---------------- epilogue: TMEM -> registers -> bias / activation -> NHWC global
        asm volatile("griddepcontrol.wait;" ::: "memory");   // bias, residual and y belong to the stream's order
        const int quarter = warp & 3;      // TMEM lanes a warp may read: 32 * (warp id mod 4)
        const int sub = (warp - 2) >> 2;   // four warps share a lane quarter and take every fourth 32-column chunk
        bool ok = true;
        int gt = 0;
        if constexpr (!kF32) if (g.prob[0].pxm) {
            // (a launch with the positions as M carries one problem; 16-bit data only)
            const TcArgs& a = g.prob[0];
            T* __restrict__ yg = reinterpret_cast<T*>(a.y);
            const uint2* pos_tab = pos_tab_all;
            // Positions are the TMEM lanes: a thread owns one position and reads its filters sixteen at a time, which
            // are contiguous in NHWC -- no transpose.  One filter tile covers the layer, so the bias is staged once.
            float* bias_s = reinterpret_cast<float*>(epi_patch);
            for (int i = threadIdx.x - 64; i < a.n_cols; i += kEpiWarps * 32)
                bias_s[i] = (a.bias && i < a.Cout) ? __ldg(a.bias + i) : 0.f;
            asm volatile("bar.sync 1, %0;" ::"n"(kEpiWarps * 32) : "memory");
            const int n_chunks = a.n_cols >> 4, items = a.MH * n_chunks;
            const bool vec_ok = (a.y_c_stride % 8 == 0) && (a.y_c_off % 8 == 0);
            int as = 0;
            unsigned pfull = 0;   // accumulator stage of this tile and the parity of its "full" phase
            for (int tile = blockIdx.x; tile < n_tiles && ok; tile += gridDim.x, ++gt, pfull ^= (as + 1 == g.AS), as = as + 1 == g.AS ? 0 : as + 1) {
                const TileIdx ti = tile_of(a, tile);
                const int n = ti.n;
                const int y0 = ti.ty * a.TH, x0 = ti.tx * a.TW;
                ok = mbar_wait(bar_accFull + 8 * as, pfull, g.wait_cycles);
                if (!ok) break;
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                const unsigned d_base = tmem_base + (unsigned)(as * g.acc_stride) + ((unsigned)(quarter * 32) << 16);
                T* yb = yg + (((size_t)n * a.Ho + y0) * a.Wo + x0) * a.y_c_stride + a.y_c_off;
                const unsigned ry = (unsigned)min(a.TH, a.Ho - y0), rx = (unsigned)min(a.TW, a.Wo - x0);
                for (int item = sub; item < items; item += 4) {
                    const int h = item / n_chunks, c = item - h * n_chunks;
                    unsigned r[16];
                    tmem_ld16(d_base + (unsigned)(h * a.n_cols + c * 16), r);
                    const uint2 e = pos_tab[h * 128 + quarter * 32 + lane];
                    const bool px_ok = (e.y >> 16) < ry && (e.y & 0xFFFFu) < rx;
                    const float* b16 = bias_s + c * 16;
                    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
                    unsigned o[8];
                    if (a.act == RTOSS_ACT_SILU) act_pack16<T, RTOSS_ACT_SILU>(r, b16, o);
                    else if (a.act == RTOSS_ACT_RELU) act_pack16<T, RTOSS_ACT_RELU>(r, b16, o);
                    else act_pack16<T, RTOSS_ACT_NONE>(r, b16, o);
                    if (px_ok) {
                        T* dst = yb + e.x + c * 16;
                        if (vec_ok && c * 16 + 16 <= a.Cout) {
                            reinterpret_cast<uint4*>(dst)[0] = make_uint4(o[0], o[1], o[2], o[3]);
                            reinterpret_cast<uint4*>(dst)[1] = make_uint4(o[4], o[5], o[6], o[7]);
                        } else {
                            // ragged filter count or unaligned channel slice: element stores
                            const T* ov = reinterpret_cast<const T*>(o);
#pragma unroll
                            for (int j = 0; j < 16; ++j)
                                if (c * 16 + j < a.Cout) dst[j] = ov[j];
                        }
                    }
                }
                asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
                __syncwarp();
                if (lane == 0) asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar_accEmpty + 8 * as) : "memory");
            }
            gt = -1;   // (done: the loop below does not run)
        }
        int pi = 0, as = 0;
        unsigned pfull = 0;   // accumulator stage of this tile and the parity of its "full" phase
        for (int tile = blockIdx.x; gt >= 0 && tile < n_tiles && ok; tile += gridDim.x, ++gt, pfull ^= (as + 1 == g.AS), as = as + 1 == g.AS ? 0 : as + 1) {
            int local;
            pi = find_problem<kMulti>(g, tile, local, pi);
            const TcArgs& a = g.prob[pi];
            T* __restrict__ yg = reinterpret_cast<T*>(a.y);
            const uint2* pos_tab = pos_tab_all + a.tab * kMaxPx;
            const unsigned s_tab = s_tab_all + (unsigned)a.tab * kMaxPx * 8;
            const TileIdx ti = tile_of(a, local);   // a unit is (tile proper, share of the channel blocks)
            const int n = ti.n;
            const int y0 = ti.ty * a.TH, x0 = ti.tx * a.TW, co0 = ti.cot * kMTile;
            // Everything that does not need the accumulator comes before the wait for it: the bias is a global load
            // (a cold one costs more than a thousand cycles) and would otherwise sit on the path of every tile.
            // TMEM lane = filter.  A narrow layer's filters are repeated down the lanes (R copies): every lane quarter
            // then holds outputs, and the copies share the tile's columns between them.
            const int copy = (quarter * 32) >> a.rep_shift, row0 = quarter * 32 - (copy << a.rep_shift);   // (rep_rows is 32, 64 or 128)
            const int co = co0 + row0 + lane;
            const bool co_ok = co < a.Cout;
            const float bv = (a.bias && co_ok) ? __ldg(a.bias + co) : 0.f;
            const unsigned patch = s_tmem_ptr + 16 + (unsigned)(warp - 2) * kPatchBytes;  // shared address
            // (fp32 outputs leave through the element stores below: a warp's 32 filters of one position are 128 contiguous bytes)
            const bool vec_ok = !kF32 && (a.y_c_stride % 8 == 0) && ((a.y_c_off + co0) % 8 == 0) && (co0 + row0 + 32 <= a.Cout);
            T* yb = yg + (((size_t)n * a.Ho + y0) * a.Wo + x0) * a.y_c_stride + a.y_c_off + co0 + row0;
            const unsigned ry = (unsigned)min(a.TH, a.Ho - y0), rx = (unsigned)min(a.TW, a.Wo - x0);  // rows / columns inside the image
            const int c_first = (sub + 4 * copy) * 32, c_step = 128 * a.R;
            const T* rb = a.resid ? reinterpret_cast<const T*>(a.resid) + (yb - yg) : nullptr;   // laid out like y
            const bool post = a.resid_post != 0;
            const float bs = (!kF32 && a.act == RTOSS_ACT_SILU && (!rb || post)) ? 0.5f * bv : bv;   // (a residual in front of the activation, or fp32 data: plain bias)
            ok = mbar_wait(bar_accFull + 8 * as, pfull, g.wait_cycles);
            if (!ok && a.KS == 1) break;   // (split K: the cluster barriers below must still be passed)
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            const unsigned d_base = tmem_base + (unsigned)(as * g.acc_stride) + ((unsigned)(quarter * 32) << 16);
            if (a.KS > 1) {
                // ---- split K.  The KS CTAs of the cluster hold the partial sums of one tile.  Barrier 1: every CTA's
                // MMAs have completed, so the operand rings of all of them are free; each CTA then stores its partial
                // sums of chunk c into the shared memory of the chunk's owner (rank c % KS); barrier 2: all stores have
                // landed; every CTA adds up and finishes the chunks it owns.  Every thread of the cluster passes both
                // barriers, whatever happened to its waits (the other roles pass them at the end of the kernel).
                const int rank = (int)cluster_rank(), n_chunks = (a.N_px + 31) >> 5, n_lc = (n_chunks + a.KS - 1) / a.KS;
                cluster_sync_all();
                if (ok) {
                    for (int c0 = c_first; c0 < a.N_px; c0 += c_step) {
                        unsigned r[32];
                        tmem_ld32(d_base + (unsigned)c0, r);
                        asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
                        const int c = c0 >> 5;
                        const unsigned dst = peer_smem(sA + (unsigned)((((rank * n_lc + c / a.KS) * 32) * 128 + quarter * 32 + lane) * 4),
                                                       (unsigned)(c % a.KS));
#pragma unroll
                        for (int j = 0; j < 32; ++j) st_peer_f32(dst + j * 512, __uint_as_float(r[j]));   // 128 contiguous bytes per warp
                    }
                }
                asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
                cluster_sync_all();
                if (ok) {
                    const int row = quarter * 32 + lane;
                    if (a.act == RTOSS_ACT_SILU)
                        epilogue_from_shares<T, RTOSS_ACT_SILU>(sA, a.KS, rank, n_lc, sub, row, a.N_px, bs, vec_ok, co_ok, patch, s_tab, pos_tab, yb, ry, rx, lane, rb, post);
                    else if (a.act == RTOSS_ACT_RELU)
                        epilogue_from_shares<T, RTOSS_ACT_RELU>(sA, a.KS, rank, n_lc, sub, row, a.N_px, bs, vec_ok, co_ok, patch, s_tab, pos_tab, yb, ry, rx, lane, rb, post);
                    else
                        epilogue_from_shares<T, RTOSS_ACT_NONE>(sA, a.KS, rank, n_lc, sub, row, a.N_px, bs, vec_ok, co_ok, patch, s_tab, pos_tab, yb, ry, rx, lane, rb, post);
                }
                continue;
            }
            bool stored = false;
            if constexpr (!kF32) {
                if (vec_ok) {
                    stored = true;
                    if (rb) {
                        const unsigned stage = s_res + (unsigned)(warp - 2) * kResStage;
#define RTOSS_RES_CALL(ACT_, POST_) \
        epilogue_chunks_res<T, ACT_, POST_>(d_base, c_first, c_step, a.N_px, bs, patch, s_tab, yb, ry, rx, lane, rb, stage)
                        if (post) {
                            if (a.act == RTOSS_ACT_SILU) RTOSS_RES_CALL(RTOSS_ACT_SILU, true);
                            else if (a.act == RTOSS_ACT_RELU) RTOSS_RES_CALL(RTOSS_ACT_RELU, true);
                            else RTOSS_RES_CALL(RTOSS_ACT_NONE, false);   // no activation: both orders are the same sum
                        } else {
                            if (a.act == RTOSS_ACT_SILU) RTOSS_RES_CALL(RTOSS_ACT_SILU, false);
                            else if (a.act == RTOSS_ACT_RELU) RTOSS_RES_CALL(RTOSS_ACT_RELU, false);
                            else RTOSS_RES_CALL(RTOSS_ACT_NONE, false);
                        }
#undef RTOSS_RES_CALL
                    } else if (a.act == RTOSS_ACT_SILU)
                        epilogue_chunks<T, RTOSS_ACT_SILU>(d_base, c_first, c_step, a.N_px, bs, patch, s_tab, yb, ry, rx, lane, rb);
                    else if (a.act == RTOSS_ACT_RELU)
                        epilogue_chunks<T, RTOSS_ACT_RELU>(d_base, c_first, c_step, a.N_px, bs, patch, s_tab, yb, ry, rx, lane, rb);
                    else
                        epilogue_chunks<T, RTOSS_ACT_NONE>(d_base, c_first, c_step, a.N_px, bs, patch, s_tab, yb, ry, rx, lane, rb);
                }
            }
            if (!stored) {
                // ragged filter counts, unaligned channel slices, fp32 data: element stores, lane = filter
                for (int c0 = c_first; c0 < a.N_px; c0 += c_step) {
                    unsigned r[32];
                    tmem_ld32(d_base + (unsigned)c0, r);
                    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
                    for (int j = 0; j < 32; ++j) {
                        const uint2 e = pos_tab[c0 + j];
                        const bool in_img = co_ok && (e.y >> 16) < ry && (e.y & 0xFFFFu) < rx;
                        float v = __uint_as_float(r[j]) + bv;
                        if (rb && in_img && !post) v = to_f32<T>(from_f32<T>(v)) + to_f32<T>(__ldcg(rb + e.x + lane));   // round, then add the residual
                        if (a.act == RTOSS_ACT_RELU) v = fmaxf(v, 0.f);
                        if (a.act == RTOSS_ACT_SILU) {
                            if (kF32) {
                                v = silu_f32(v);
                            } else {
                                float th;
                                asm("tanh.approx.f32 %0, %1;" : "=f"(th) : "f"(0.5f * v));
                                v = v * fmaf(0.5f, th, 0.5f);
                            }
                        }
                        if (rb && in_img && post) v = to_f32<T>(from_f32<T>(v)) + to_f32<T>(__ldcg(rb + e.x + lane));   // behind the activation
                        if (co_ok && (e.y >> 16) < ry && (e.y & 0xFFFFu) < rx) yb[e.x + lane] = from_f32<T>(v);
                    }
                }
            }
            // this warp has read everything it needs from the accumulator stage
            asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
            __syncwarp();
            if (lane == 0) asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar_accEmpty + 8 * as) : "memory");
            if (kMulti && g.done && tile + (int)gridDim.x >= g.unit_end[pi]) {
                // This was the CTA's last tile of the problem: the warp reports its share of the outputs written.  The
                // lanes' stores are ordered before lane 0's fence by the __syncwarp above, the fence before the count.
                if (lane == 0) {
                    __threadfence();
                    atomicAdd(g.done + pi, 1u);
                }
            }
        }
        if (!ok && lane == 0) atomicExch(g.status, 3);
    }

    if (g.prob[0].KS > 1 && (warp < 2 || warp >= kWeightWarp)) {   // (a launch cut along K carries one problem)   // split K: the barriers the epilogue warps pass around the exchange
        cluster_sync_all();
        cluster_sync_all();
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (warp == 1) {
        __syncwarp();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(g.tmem_cols) : "memory");
    }
    if (kMulti && g.done && threadIdx.x == 0) {
        // The completion counters go back to zero for the next launch: by the last CTA to get here, when no CTA of this
        // launch reads them any more.
        __threadfence();
        if (atomicAdd(g.done + kMaxProb, 1u) == gridDim.x - 1) {
            for (int i = 0; i <= kMaxProb; ++i) g.done[i] = 0u;
        }
    }
}

PFN_cuTensorMapEncodeTiled_v12000 encode_fn() {
    static PFN_cuTensorMapEncodeTiled_v12000 fn = nullptr;
    static bool tried = false;
    if (!tried) {
        tried = true;
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<PFN_cuTensorMapEncodeTiled_v12000>(p);
    }
    return fn;
}

inline int round_up(int v, int m) { return (v + m - 1) / m * m; }

// Which operand the positions are.  A tcgen05.mma costs about the same whatever its N, so the wide operand should be
// N: with the filters as M and up to 256 positions as N a layer of 128 filters per tile runs near the tensor peak.
// A narrow layer wastes most of M that way and, worse, leaves three of four epilogue warps without TMEM lanes to
// read; with the positions as M every lane carries an output and a thread's filters are contiguous in NHWC.  The
// price is one instruction per 128 positions instead of per 256: taken where few instructions are needed anyway.
bool use_pxm(const rtoss_packed* p) { return p->Cout <= kPxmMaxCout && p->ksize == 1 && p->dtype != RTOSS_F32; }

// Bytes of a staged row: 16-bit layers of at most 32 input channels stage 64-byte rows (64-byte swizzle) instead of
// 128-byte rows half of which would be zero fill.
int row_bytes_of(const rtoss_packed* p) { return (p->dtype != RTOSS_F32 && p->Cin <= 32) ? 64 : kRowBytes; }
// channel blocks (staged rows' worth of channels) of a layer
int ncb_of(const rtoss_packed* p) {
    const int cb_ch = row_bytes_of(p) / (p->dtype == RTOSS_F32 ? 4 : 2);
    return (p->Cin + cb_ch - 1) / cb_ch;
}

struct TcPlan {
    int TH, TW, Wq, N_px, NA, NB, G, n_sub, sub_rows, rows_staged, tiles_x, smem;
};

// Geometry of a tile.  Positions of a tile run over TH rows of pitch Wq = TW + (columns of halo the
// staged rows carry); every tap reads the staged list from a shifted start row.
//   3x3 stride 1: one staged tile, TH+2 rows of TW+2 pixels, tap (r,c) at shift r*Wq + c.
//   1x1:          one staged tile, TH rows of TW pixels (stride 2: every second pixel and row, picked by
//                 the TMA element strides), shift 0.
//   3x3 stride 2: four staged tiles, one per (row parity, column parity) of the input, each TH+1 rows of
//                 TW+1 pixels fetched with element strides 2; tap r reads the odd rows for r = 0, 2 and
//                 the even rows for r = 1, one staged row further down for r = 1, 2; columns alike.
// The plan picks TH, the column segment TW (images wider than a TMA box are cut into segments), the
// ring depths, and how many taps share a weight stage.
bool plan_tc(int N, int Ho, int Wo, int ksize, int S, int co_tiles, int sm_count, bool pxm, int w_rows, bool resid, TcPlan* out,
             int n_prob = 1, bool f32 = false, int force_G = 0, int n_tabs = 1, int row_bytes = kRowBytes, int ncb = 2) {
    const int halo = ksize == 3 ? (S == 1 ? 2 : 1) : 0;
    const int n_sub = (ksize == 3 && S == 2) ? 4 : 1;
    const int max_pitch = S == 1 ? 256 : 128;  // TMA box: at most 256 elements traversed per dimension
    const int fixed = 1024 /*alignment slack*/ + 512 /*barriers*/ + kEpiWarps * kPatchBytes /*epilogue patches*/ +
                      n_tabs * kMaxPx * 8 /*position tables*/ + (resid ? kEpiWarps * kResStage : 0) /*staging of the residual operand*/;
    const int cap = 227 * 1024 - 64;
    const bool grouped = n_prob > 1;   // one of several problems that run side by side: together they fill the SMs
    double best = -1;
    for (int nseg = 1; nseg <= 16; ++nseg) {
        const int tw = (Wo + nseg - 1) / nseg;
        const int wq = tw + halo;
        if (wq > max_pitch || wq > 256) continue;
        for (int th = 1; th <= Ho; ++th) {
            const int rows_staged = th + halo;
            if (th * wq > 256 || rows_staged * S > 256) break;
            const int n_px = round_up(th * wq, 16);
            const int max_shift = ksize == 3 ? (S == 1 ? 2 * wq + 2 : wq + 1) : 0;
            int need_rows = n_px + max_shift > rows_staged * wq ? n_px + max_shift : rows_staged * wq;
            // positions as the M operand: every instruction reads 128 rows, also where the tile's list ends earlier
            const int halves = n_px > 128 ? 2 : 1;
            if (pxm && max_shift + 128 * halves > need_rows) need_rows = max_shift + 128 * halves;
            const int sub_rows = round_up(need_rows, 8);
            const int a_bytes = n_sub * sub_rows * row_bytes * (f32 ? 2 : 1);   // (fp32: heads and remainders)
            for (int G = (ksize == 3 ? 3 : 1); G >= 1; G -= 2) {
                if (force_G && G != force_G) continue;   // (the problems of one launch share the weight ring: one G for all)
                const int b_bytes = G * w_rows * row_bytes;
                int na = (cap - fixed - 2 * b_bytes) / a_bytes;
                if (na < 1) continue;
                if (na > kMaxA) na = kMaxA;
                // A channel block feeds nine taps: with several blocks per tile two stages cover the load.  A layer of
                // one block per tile (at most 64 channels; 32 with 64-byte rows) has the next TILE's block as its next
                // stage, and its instructions (18 or 36 of at most 128 cycles) are over before a fetch from L2 returns:
                // it keeps as many stages as fit.
                if (na > 2 && ksize == 3 && ncb > 1) na = 2;
                int nb = (cap - fixed - na * a_bytes) / b_bytes;
                if (nb > kMaxB) nb = kMaxB;
                if (nb < 2) continue;
                const long tiles = (long)N * ((Ho + th - 1) / th) * nseg * co_tiles;
                const double waves = (double)tiles / sm_count;
                const double balance = grouped ? 1.0 : waves / (double)((tiles + sm_count - 1) / sm_count);  // 1 = SMs equally loaded
                // What counts is useful positions per tensor-pipe cycle.  An instruction with the filters on M and N positions
                // takes N / 2 cycles, but never less than 76 (measured: 128.2 cycles at N = 256, 75.9 at every N <= 128).
                // That is the measure for 3x3 layers of stride 1, whose tiles are bound by their instructions; the tiles of
                // 1x1 and stride-2 layers are bound by what surrounds the instructions (fetches, barrier rounds, the
                // epilogue) and do better with as many positions per tile as fit (measured both ways, layer by layer).
                // (Nor does it pay where the smaller tiles would still fit one wave: such layers gain more from tiles of 256
                // positions cut along the channel blocks.)
                const bool by_cycles = ksize == 3 && S == 1 && n_px / 2.0 < 128.0 && (grouped || tiles > sm_count);
                const double instr_cycles = pxm ? 128.0 * halves : by_cycles ? (n_px / 2.0 > 76.0 ? n_px / 2.0 : 76.0) : 128.0;
                const double eff = (double)(th * tw) / (2.0 * instr_cycles) * Ho / (double)((Ho + th - 1) / th * th) * Wo / (double)(tw * nseg);
                const double halo_cost = (double)(th * tw) / (double)(rows_staged * wq);  // staged pixels that are outputs
                // (fp32: a block feeds 108 instructions, twelve per tap, so a stage per tap costs little, while a single
                // activation stage leaves the fetch and the split of the next block uncovered)
                const double score = eff * (0.5 + 0.5 * balance) * (G == 3 || ksize == 1 ? 1.0 : (f32 ? 0.95 : 0.8)) *
                                         (na >= 2 ? 1.0 : (f32 ? 0.7 : 0.8)) * (0.8 + 0.2 * halo_cost) +
                                     1e-4 * th;
                if (score > best) {
                    best = score;
                    out->TH = th;
                    out->TW = tw;
                    out->Wq = wq;
                    out->N_px = n_px;
                    out->NA = na;
                    out->NB = nb;
                    out->G = G;
                    out->n_sub = n_sub;
                    out->sub_rows = sub_rows;
                    out->rows_staged = rows_staged;
                    out->tiles_x = nseg;
                    out->smem = na * a_bytes + nb * b_bytes + fixed;
                }
                if (!f32) break;  // 16-bit data: the largest G that fits is taken for this (th, tw); fp32 weighs both
            }
        }
    }
    return best > 0;
}

// What one problem adds to a launch besides its TcArgs.
struct ProbPlan {
    TcPlan plan;
    int a_stage_bytes, b_stage_bytes, acc_cols;
};

// Geometry, operand roles and TMA descriptors of one convolution.  The rings' depths and the split along K are the
// launch's business (the caller's).  Returns a cudaError_t as int.
int build_problem(const rtoss_ctx* ctx, const rtoss_packed* p, const void* x, void* y, const rtoss_conv_desc* d, int n_prob, int sms,
                  TcArgs* out, ProbPlan* pp, CUtensorMap* tmA_out, CUtensorMap* tmB_out, int force_G = 0, int n_tabs = 1) {
    const int taps = p->ksize == 3 ? 9 : 1;
    const int S = d->stride;
    const int Ho = (d->H - 1) / S + 1, Wo = (d->W - 1) / S + 1;
    const int N_T = kMTile;
    TcPlan& plan = pp->plan;
    // narrow layers put the positions on the M operand (all 128 TMEM lanes carry outputs whatever Cout is)
    const bool pxm = use_pxm(p);
    const int w_rows = pxm ? round_up(p->Cout, 16) : kMTile;
    const bool f32 = p->dtype == RTOSS_F32;
    const int esize = f32 ? 4 : 2;
    const int row_bytes = row_bytes_of(p);
    if (!plan_tc(d->N, Ho, Wo, p->ksize, S, (p->Cout + kMTile - 1) / kMTile, sms, pxm, w_rows, d->residual_dev != nullptr, &plan, n_prob, f32,
                 force_G, n_tabs, row_bytes, (p->Cin + row_bytes / esize - 1) / (row_bytes / esize)))
        return (int)cudaErrorInvalidConfiguration;

    TcArgs& a = *out;
    memset(&a, 0, sizeof(a));
    a.y = y;
    a.resid = d->residual_dev;
    a.resid_post = (d->residual_dev && d->residual_after_act) ? 1 : 0;
    a.bias = d->bias_dev;
    a.issue = p->ksize == 3 ? p->issue : nullptr;
    a.N = d->N;
    a.Ho = Ho;
    a.Wo = Wo;
    a.S = S;
    a.Cin = p->Cin;
    a.Cout = p->Cout;
    a.Wq = plan.Wq;
    a.TH = plan.TH;
    a.TW = plan.TW;
    a.taps = taps * (f32 ? 2 : 1);   // weight tiles per channel block: fp32 has the heads, then the remainders
    a.taps_real = taps;
    a.row_bytes = row_bytes;
    a.desc_hi = (unsigned)(make_sw_desc(0, row_bytes) >> 32);
    a.cb_ch = row_bytes / esize;
    a.slab_ch = 32 / esize;
    a.tiles_x = plan.tiles_x;
    a.n_sub = plan.n_sub;
    a.sub_bytes = plan.sub_rows * row_bytes;
    if (p->ksize == 3 && S == 1) {
        a.x_add[0] = a.y_add[0] = -1;
        for (int t = 0; t < 9; ++t) a.tap_shift[t] = (t / 3) * plan.Wq + (t % 3);
    } else if (p->ksize == 3) {
        // sub-tile index = 2*(row parity) + (column parity); parity 0 = even input rows / columns
        for (int sub = 0; sub < 4; ++sub) {
            a.y_add[sub] = (sub >> 1) ? -1 : -2;
            a.x_add[sub] = (sub & 1) ? -1 : -2;
        }
        for (int t = 0; t < 9; ++t) {
            const int r = t / 3, c = t % 3;
            a.tap_sub[t] = 2 * (r == 1 ? 0 : 1) + (c == 1 ? 0 : 1);
            a.tap_shift[t] = (r == 0 ? 0 : 1) * plan.Wq + (c == 0 ? 0 : 1);
        }
    }
    a.N_px = plan.N_px;
    a.ncb = (p->Cin + a.cb_ch - 1) / a.cb_ch;
    a.tiles_y = (Ho + plan.TH - 1) / plan.TH;
    a.co_tiles = (p->Cout + N_T - 1) / N_T;
    a.lo_off = f32 ? plan.n_sub * plan.sub_rows * row_bytes : 0;
    pp->a_stage_bytes = plan.n_sub * plan.sub_rows * row_bytes * (f32 ? 2 : 1);
    a.w_rows = w_rows;
    // narrow 3x3 layers keep the filters on M and repeat them down the 128 rows of the tile
    const rtoss_wtc_layout lay = rtoss_wtc_layout_of(p->Cout, p->ksize);  // how rtoss_pack laid the weights out
    a.rep_rows = lay.copies > 1 ? lay.rep_rows : 128;
    a.R = lay.copies;
    a.rep_shift = a.rep_rows == 32 ? 5 : a.rep_rows == 64 ? 6 : 7;
    pp->b_stage_bytes = plan.G * w_rows * row_bytes;
    a.G = plan.G;
    pp->acc_cols = round_up(plan.N_px, 32);  // the epilogue reads 32 columns at a time
    a.a_tx_bytes = (unsigned)(row_bytes * plan.Wq * plan.rows_staged);  // per sub-tile
    a.b_tx_bytes = (unsigned)(row_bytes * w_rows);
    a.act = (int)d->act;
    a.y_c_off = d->y_channel_offset;
    a.y_c_stride = d->y_channel_stride ? d->y_channel_stride : p->Cout;
    a.is_bf16 = p->dtype == RTOSS_BF16;
    // instruction descriptor: fp32 accumulate, A and B of the io type (f16 0, bf16 1; kind::tf32: tf32 2), both K-major,
    // N/8 and M/16
    const unsigned fmt = f32 ? 2u : a.is_bf16 ? 1u : 0u;
    a.idesc = (1u << 4) | (fmt << 7) | (fmt << 10) | ((unsigned)(plan.N_px >> 3) << 17) | ((unsigned)(kMTile >> 4) << 24);
    a.pxm = pxm ? 1 : 0;
    a.MH = plan.N_px > 128 ? 2 : 1;
    a.n_cols = round_up(p->Cout, 16);
    if (pxm) {
        pp->acc_cols = round_up(a.MH * a.n_cols, 32);
        a.idesc = (1u << 4) | (fmt << 7) | (fmt << 10) | ((unsigned)(a.n_cols >> 3) << 17) | ((unsigned)(128 >> 4) << 24);
    }
    a.KS = 1;
    a.cb_per = a.ncb;
    magic_of(a.KS, a.div_ks);
    magic_of(pxm ? 1 : a.co_tiles, a.div_co);   // (positions on M: one filter tile covers the layer)
    magic_of(a.tiles_x, a.div_tx);
    magic_of(a.tiles_y, a.div_ty);

    PFN_cuTensorMapEncodeTiled_v12000 enc = encode_fn();
    if (!enc) return (int)cudaErrorNotSupported;
    const CUtensorMapDataType dt = f32 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT32 : a.is_bf16 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_FLOAT16;
    // activations: descriptor cached per (pointer, shape, box)
    const int key[6] = {d->N, d->H, d->W, p->Cin, plan.rows_staged * 8 + S, plan.Wq * 4 + (int)p->dtype};   // (row size: a function of Cin and dtype)
    rtoss_tmap_entry* ea = nullptr;
    for (rtoss_tmap_entry& e : ctx->tmap_cache)
        if (e.valid && e.base == x && memcmp(e.dims, key, sizeof(key)) == 0) ea = &e;
    if (!ea) {
        ea = &ctx->tmap_cache[ctx->tmap_next];
        ctx->tmap_next = (ctx->tmap_next + 1) % 32;
        cuuint64_t dims[4] = {(cuuint64_t)p->Cin, (cuuint64_t)d->W, (cuuint64_t)d->H, (cuuint64_t)d->N};
        cuuint64_t strides[3] = {(cuuint64_t)p->Cin * esize, (cuuint64_t)d->W * p->Cin * esize, (cuuint64_t)d->H * d->W * p->Cin * esize};
        // with element strides the box is counted in traversed elements: S*n covers n fetched pixels
        cuuint32_t box[4] = {(cuuint32_t)a.cb_ch, (cuuint32_t)(plan.Wq * S), (cuuint32_t)(plan.rows_staged * S), 1};
        cuuint32_t es[4] = {1, (cuuint32_t)S, (cuuint32_t)S, 1};
        ea->valid = 0;
        CUresult r = enc(reinterpret_cast<CUtensorMap*>(ea->map), dt, 4, const_cast<void*>(x), dims, strides, box, es,
                         CU_TENSOR_MAP_INTERLEAVE_NONE, row_bytes == 64 ? CU_TENSOR_MAP_SWIZZLE_64B : CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                         CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
        if (r != CUDA_SUCCESS) return (int)cudaErrorInvalidValue;
        ea->base = x;
        memcpy(ea->dims, key, sizeof(key));
        ea->valid = 1;
    }
    // weights: one descriptor per handle
    rtoss_tmap_entry* eb = &p->wtc_map;
    if (!eb->valid || eb->base != p->wtc || eb->dims[0] != w_rows || eb->dims[1] != plan.G) {
        cuuint64_t dims[3] = {(cuuint64_t)p->Cin, (cuuint64_t)lay.rows, (cuuint64_t)a.taps};
        cuuint64_t strides[2] = {(cuuint64_t)p->Cin * esize, (cuuint64_t)lay.rows * p->Cin * esize};
        cuuint32_t box[3] = {(cuuint32_t)a.cb_ch, (cuuint32_t)w_rows, (cuuint32_t)plan.G};  // a weight stage is one copy
        cuuint32_t es[3] = {1, 1, 1};
        eb->valid = 0;
        CUresult r = enc(reinterpret_cast<CUtensorMap*>(eb->map), dt, 3, p->wtc, dims, strides, box, es,
                         CU_TENSOR_MAP_INTERLEAVE_NONE, row_bytes == 64 ? CU_TENSOR_MAP_SWIZZLE_64B : CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                         CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
        if (r != CUDA_SUCCESS) return (int)cudaErrorInvalidValue;
        eb->base = p->wtc;
        eb->dims[0] = w_rows;
        eb->dims[1] = plan.G;
        eb->valid = 1;
    }
    memcpy(tmA_out, ea->map, sizeof(CUtensorMap));
    memcpy(tmB_out, eb->map, sizeof(CUtensorMap));
    return 0;
}

// Split K where the layer has too few tiles for the SMs and several channel blocks: a tile's MMAs are one serial chain
// (an instruction costs the same however few positions it covers), so the blocks go to several CTAs.  The exchange
// costs a few thousand cycles (two cluster barriers, 128 KB through distributed shared memory): chains of 72
// instructions (3x3: two channel blocks) resp. 32 (1x1: eight blocks) and more are cut, a share keeps at least one
// block (1x1: two); cutting shorter 1x1 chains was measured and lost.  The CTAs of a tile form one cluster (at most
// 8), one CTA per share.  *ks = 1 leaves the layer uncut.
void pick_split(int ksize, bool pxm, int R, long tiles, int ncb, int n_px, int rings, int sms, int* ks_out, int* cb_per_out) {
    *ks_out = 1;
    *cb_per_out = ncb;
    const int min_cb = ksize == 3 ? 1 : 2;
    const int min_ncb = ksize == 3 ? 2 : 8;
    const int n_lc_max = 8;   // a tile has at most 8 chunks of 32 columns: the owner's buffers take KS * ceil(chunks / KS) * 16 KB
    if (pxm || R != 1 || tiles * 2 > sms || ncb < min_ncb) return;
    int want = (int)(sms / tiles);
    if (want > ncb / min_cb) want = ncb / min_cb;
    if (want > 8) want = 8;
    while (want > 1) {
        const int cb_per = (ncb + want - 1) / want, ks = (ncb + cb_per - 1) / cb_per;
        const int n_chunks = (n_px + 31) / 32, n_lc = (n_chunks + ks - 1) / ks;
        if (ks > 1 && ks * n_lc <= 2 * n_lc_max && (size_t)ks * n_lc * 16384 <= (size_t)rings) {
            *cb_per_out = cb_per;
            *ks_out = ks;
            return;
        }
        --want;
    }
}

// Both instantiations may use up to the whole shared memory of an SM; the attribute belongs to the (function, device)
// pair, so there is one flag per device.
int ensure_smem_attr(const rtoss_ctx* ctx) {
    static std::atomic<bool> attr_set[64];
    const int dev_slot = ctx->device >= 0 && ctx->device < 64 ? ctx->device : -1;
    if (dev_slot < 0 || !attr_set[dev_slot].load(std::memory_order_acquire)) {
        cudaError_t e = cudaFuncSetAttribute(conv_tc_kernel<__nv_bfloat16, TcLaunch1>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024);
        if (e == cudaSuccess)
            e = cudaFuncSetAttribute(conv_tc_kernel<__half, TcLaunch1>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024);
        if (e == cudaSuccess)
            e = cudaFuncSetAttribute(conv_tc_kernel<__nv_bfloat16, TcLaunchN>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024);
        if (e == cudaSuccess)
            e = cudaFuncSetAttribute(conv_tc_kernel<__half, TcLaunchN>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024);
        if (e == cudaSuccess)
            e = cudaFuncSetAttribute(conv_tc_kernel<float, TcLaunch1>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024);
        if (e == cudaSuccess)
            e = cudaFuncSetAttribute(conv_tc_kernel<float, TcLaunchN>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024);
        if (e != cudaSuccess) return (int)e;
        if (dev_slot >= 0) attr_set[dev_slot].store(true, std::memory_order_release);
    }
    return 0;
}

template <typename G>
void launch_common(const rtoss_ctx* ctx, G* g) {
    g->status = ctx->dev_status;
    g->wait_cycles = ctx->wait_cycles > 0 ? ctx->wait_cycles : kWaitCycles;
    g->inject = 0;
    g->AS = 2;
    int alloc = 32;
    while (alloc < g->AS * g->acc_stride) alloc <<= 1;
    g->tmem_cols = alloc;
}

}  // namespace

bool rtoss_tc_weights_eligible(const rtoss_packed* p) {
    return ((p->dtype == RTOSS_BF16 || p->dtype == RTOSS_F16) && p->Cin % 8 == 0) || (p->dtype == RTOSS_F32 && p->Cin % 4 == 0);  // 16-byte rows for TMA
}

// Can this call run on the tensor path?
bool rtoss_tc_eligible(const rtoss_packed* p, const rtoss_conv_desc* d, const void* x, const void* y) {
    if (!p->wtc || !rtoss_tc_weights_eligible(p)) return false;
    if (d->layout != RTOSS_NHWC || (int)d->io_dtype != (int)p->dtype) return false;
    if ((reinterpret_cast<uintptr_t>(x) & 15) || (reinterpret_cast<uintptr_t>(y) & 15)) return false;
    if (!encode_fn()) return false;
    // a residual operand: 16-byte aligned, and not for the positions-as-M form (narrow 1x1 layers)
    if (d->residual_dev && (use_pxm(p) || (reinterpret_cast<uintptr_t>(d->residual_dev) & 15))) return false;
    const int Ho = (d->H - 1) / d->stride + 1, Wo = (d->W - 1) / d->stride + 1;
    TcPlan plan;
    const bool pxm = use_pxm(p);
    return plan_tc(d->N, Ho, Wo, p->ksize, d->stride, (p->Cout + kMTile - 1) / kMTile, 148, pxm, pxm ? round_up(p->Cout, 16) : kMTile,
                   d->residual_dev != nullptr, &plan, 1, p->dtype == RTOSS_F32, 0, 1, row_bytes_of(p), ncb_of(p));
}

// May this call be one of several in a launch?  (Tensor path with the filters on M.)
bool rtoss_tc_groupable(const rtoss_packed* p, const rtoss_conv_desc* d, const void* x, const void* y) {
    return !use_pxm(p) && rtoss_tc_eligible(p, d, x, y);
}

// Would a launch of its own cut this call along K (few tiles, many channel blocks)?  Such a call is faster alone than
// as a member of a shared launch, which never cuts -- unless the other members keep the SMs busy meanwhile.
// *tiles_out (nullable): the call's tiles of 128 filters.
bool rtoss_tc_prefers_split(const rtoss_ctx* ctx, const rtoss_packed* p, const rtoss_conv_desc* d, long* tiles_out) {
    const int sms = ctx->sm_count > 0 ? ctx->sm_count : 148;
    const int Ho = (d->H - 1) / d->stride + 1, Wo = (d->W - 1) / d->stride + 1;
    const bool pxm = use_pxm(p), f32 = p->dtype == RTOSS_F32;
    const int w_rows = pxm ? round_up(p->Cout, 16) : kMTile, co_tiles = (p->Cout + kMTile - 1) / kMTile;
    TcPlan plan;
    if (tiles_out) *tiles_out = 0;
    const int row_bytes = row_bytes_of(p);
    if (!plan_tc(d->N, Ho, Wo, p->ksize, d->stride, co_tiles, sms, pxm, w_rows, d->residual_dev != nullptr, &plan, 1, f32, 0, 1, row_bytes, ncb_of(p))) return false;
    const int a_stage = plan.n_sub * plan.sub_rows * row_bytes * (f32 ? 2 : 1), b_stage = plan.G * w_rows * row_bytes;
    const int cb_ch = row_bytes / (f32 ? 4 : 2);
    const long tiles = (long)d->N * ((Ho + plan.TH - 1) / plan.TH) * plan.tiles_x * co_tiles;
    if (tiles_out) *tiles_out = tiles;
    int ks = 1, cb_per = 0;
    pick_split(p->ksize, pxm, rtoss_wtc_layout_of(p->Cout, p->ksize).copies, tiles, (p->Cin + cb_ch - 1) / cb_ch, plan.N_px,
               plan.NA * a_stage + plan.NB * b_stage, sms, &ks, &cb_per);
    return ks > 1;
}

extern "C" rtoss_status rtoss_tensor_plan_of(const rtoss_conv_desc* d, int ksize, int Cin, int Cout, rtoss_dtype dtype, int sm_count,
                                            rtoss_tensor_plan* out) {
    if (!d || !out || (ksize != 1 && ksize != 3) || Cin < 1 || Cout < 1 || (int)dtype < 0 || (int)dtype > 2 || d->N < 1 || d->H < 1 ||
        d->W < 1 || (d->stride != 1 && d->stride != 2))
        return RTOSS_ERR_INVALID_ARG;
    memset(out, 0, sizeof(*out));
    rtoss_packed fake;
    memset(&fake, 0, sizeof(fake));
    fake.Cin = Cin, fake.Cout = Cout, fake.ksize = ksize, fake.dtype = dtype;
    const rtoss_packed* p = &fake;
    if (!rtoss_tc_weights_eligible(p) || d->layout != RTOSS_NHWC) return RTOSS_OK;   // (eligible stays 0)
    const int sms = sm_count > 0 ? sm_count : 148;
    const int Ho = (d->H - 1) / d->stride + 1, Wo = (d->W - 1) / d->stride + 1;
    const bool pxm = use_pxm(p), f32 = dtype == RTOSS_F32;
    const int w_rows = pxm ? round_up(Cout, 16) : kMTile, co_tiles = (Cout + kMTile - 1) / kMTile;
    const int row_bytes = row_bytes_of(p);
    TcPlan plan;
    const int ncb = (Cin + row_bytes / (f32 ? 4 : 2) - 1) / (row_bytes / (f32 ? 4 : 2));
    if (!plan_tc(d->N, Ho, Wo, ksize, d->stride, co_tiles, sms, pxm, w_rows, d->residual_dev != nullptr, &plan, 1, f32, 0, 1, row_bytes, ncb))
        return RTOSS_OK;
    out->eligible = 1;
    out->rows_per_tile = plan.TH, out->cols_per_tile = plan.TW, out->pitch = plan.Wq, out->positions = plan.N_px;
    out->act_stages = plan.NA, out->weight_stages = plan.NB, out->taps_per_weight_stage = plan.G;
    out->row_bytes = row_bytes;
    out->act_stage_bytes = plan.n_sub * plan.sub_rows * row_bytes * (f32 ? 2 : 1);
    out->weight_stage_bytes = plan.G * w_rows * row_bytes;
    out->staged_rows = plan.rows_staged, out->sub_tiles = plan.n_sub;
    out->shared_bytes = plan.smem;
    out->positions_on_m = pxm ? 1 : 0;
    const long tiles = (long)d->N * ((Ho + plan.TH - 1) / plan.TH) * plan.tiles_x * (pxm ? 1 : co_tiles);
    out->tiles = (int)(tiles > 0x7FFFFFFF ? 0x7FFFFFFF : tiles);
    int ks = 1, cb_per = 0;
    pick_split(ksize, pxm, rtoss_wtc_layout_of(Cout, ksize).copies, tiles, ncb, plan.N_px,
               plan.NA * out->act_stage_bytes + plan.NB * out->weight_stage_bytes, sms, &ks, &cb_per);
    out->split_k = ks;
    return RTOSS_OK;
}

int rtoss_launch_conv_tc(const rtoss_ctx* ctx, const rtoss_packed* p, const void* x, void* y, const rtoss_conv_desc* d,
                         void* stream) {
    const int sms = ctx->sm_count > 0 ? ctx->sm_count : 148;
    static thread_local TcLaunch1 g;   // several KB: kept off the stack
    ProbPlan pp;
    g.n_prob = 1;
    int e = build_problem(ctx, p, x, y, d, 1, sms, &g.prob[0], &pp, &g.tmA[0], &g.tmB[0]);
    if (e) return e;
    TcArgs& a = g.prob[0];
    const TcPlan& plan = pp.plan;
    const bool f32 = p->dtype == RTOSS_F32;
    a.NA = plan.NA;
    a.NB = plan.NB;
    a.a_stage = (unsigned)pp.a_stage_bytes;
    a.b_stage = (unsigned)pp.b_stage_bytes;
    a.sB_off = (unsigned)plan.NA * a.a_stage;
    const int rings = (int)(a.sB_off + (unsigned)plan.NB * a.b_stage);
    g.res_off = rings;   // the staging of a residual operand lies behind the rings
    g.ring_bytes = rings + (d->residual_dev ? kEpiWarps * kResStage : 0);
    g.max_na = plan.NA;
    g.max_nb = plan.NB;
    g.n_tabs = 1;
    g.done = nullptr;
    g.acc_stride = pp.acc_cols;
    launch_common(ctx, &g);
    pick_split(p->ksize, a.pxm != 0, a.R, (long)d->N * a.tiles_y * a.tiles_x * a.co_tiles, a.ncb, plan.N_px, rings, sms, &a.KS, &a.cb_per);
    magic_of(a.KS, a.div_ks);
    // at least half an SM's shared memory, so that a second CTA (which would wait for TMEM) never shares the SM
    const size_t smem = (size_t)(plan.smem > 116 * 1024 ? plan.smem : 116 * 1024);
    size_t n_units = (size_t)d->N * a.tiles_y * a.tiles_x * a.co_tiles * a.KS;
    if (ctx->inject_next) {
        // failure-detection hook: honoured by a launch of one CTA only (every role of that CTA then runs into its
        // bounded wait and leaves through the normal exit)
        ctx->inject_next = 0;
        if (n_units != 1) return (int)cudaErrorNotSupported;
        g.inject = 1;
    }
    g.unit_end[0] = (int)n_units;
    dim3 grid((unsigned)(n_units < (size_t)sms ? n_units : (size_t)sms));
    e = ensure_smem_attr(ctx);
    if (e) return e;
    cudaError_t le;
    if (a.KS > 1) {
        // one cluster per tile; if the device cannot place the clusters the layer runs uncut
        le = f32 ? rtoss_dev::launch_pdl(conv_tc_kernel<float, TcLaunch1>, grid, kTcThreads, smem, (cudaStream_t)stream, a.KS, g)
             : a.is_bf16 ? rtoss_dev::launch_pdl(conv_tc_kernel<__nv_bfloat16, TcLaunch1>, grid, kTcThreads, smem, (cudaStream_t)stream, a.KS, g)
                         : rtoss_dev::launch_pdl(conv_tc_kernel<__half, TcLaunch1>, grid, kTcThreads, smem, (cudaStream_t)stream, a.KS, g);
        if (le == cudaSuccess) return 0;
        cudaGetLastError();
        a.KS = 1;
        magic_of(a.KS, a.div_ks);
        a.cb_per = a.ncb;
        n_units = (size_t)d->N * a.tiles_y * a.tiles_x * a.co_tiles;
        g.unit_end[0] = (int)n_units;
        grid = dim3((unsigned)(n_units < (size_t)sms ? n_units : (size_t)sms));
    }
    le = f32 ? rtoss_dev::launch_pdl(conv_tc_kernel<float, TcLaunch1>, grid, kTcThreads, smem, (cudaStream_t)stream, 1, g)
         : a.is_bf16 ? rtoss_dev::launch_pdl(conv_tc_kernel<__nv_bfloat16, TcLaunch1>, grid, kTcThreads, smem, (cudaStream_t)stream, 1, g)
                     : rtoss_dev::launch_pdl(conv_tc_kernel<__half, TcLaunch1>, grid, kTcThreads, smem, (cudaStream_t)stream, 1, g);
    return (int)le;
}

// Several convolutions in ONE launch: independent ones side by side, dependent ones one behind the other.
//
// after[i] (null: none depends on another) has bit j set when convolution i must see convolution j (j < i) complete:
// it reads what j writes, or overwrites what j reads or writes.  The kernel then keeps the CTAs that reach a tile of
// i waiting until every CTA has reported its tiles of j done (a counter per problem in device memory; the waits are
// bounded like all others).  That is only sound when all CTAs of the launch are on the device together: the grid is at
// most one CTA per SM, and nothing else may hold SMs forever while such a launch runs.
//
// All convolutions must qualify for the tensor path with the filters on M and share the data type; at most kMaxProb.
// They are sorted into levels (a convolution's level is one more than the highest level it waits for); the
// convolutions of a level with the same kernel size (and stride class, for 3x3) share one ring layout, planned as the
// grouped launches always were; a CTA that passes from one layout to another lets its rings run empty in between.
// Returns 0 after a launch, -1 when the set cannot share a launch (nothing was launched: the caller runs the calls
// one by one, in order), or a cudaError_t.
int rtoss_launch_conv_tc_chain(const rtoss_ctx* ctx, int n, const rtoss_packed* const* ps, const void* const* xs, void* const* ys,
                               const rtoss_conv_desc* const* ds, const uint32_t* after, void* stream) {
    if (n < 2 || n > kMaxProb || ctx->inject_next) return -1;
    const int sms = ctx->sm_count > 0 ? ctx->sm_count : 148;
    bool resid = false, chained = false;
    int level[kMaxProb], cls[kMaxProb];
    for (int i = 0; i < n; ++i) {
        if (use_pxm(ps[i]) || ps[i]->dtype != ps[0]->dtype) return -1;
        if (!rtoss_tc_eligible(ps[i], ds[i], xs[i], ys[i])) return -1;
        resid = resid || ds[i]->residual_dev != nullptr;
        level[i] = 0;
        if (after && after[i]) {
            if (i == 0 || (after[i] >> i)) return (int)cudaErrorInvalidValue;   // only earlier convolutions may be named
            chained = true;
            for (int j = 0; j < i; ++j)
                if ((after[i] >> j) & 1u) level[i] = level[j] + 1 > level[i] ? level[j] + 1 : level[i];
        }
        cls[i] = ps[i]->ksize == 3 ? 3 + ds[i]->stride : 1;   // 1x1 (any stride), 3x3 stride 1, 3x3 stride 2
    }
    if (chained && !ctx->chain_done) return -1;
    static thread_local TcLaunchN g;
    static thread_local TcArgs args[kMaxProb];
    static thread_local CUtensorMap mapA[kMaxProb], mapB[kMaxProb];
    ProbPlan pp[kMaxProb];
    long n_tiles[kMaxProb];
    int geo_of[kMaxProb];
    struct Geo {
        int a, b, na, nb;
        bool under;   // planned below the staging area of residual operands
    } geos[kMaxProb];
    int n_geo = 0, acc_max = 0, n_tabs_planned = 0;
    const int cap = 227 * 1024 - 64;
    const int res_bytes = resid ? kEpiWarps * kResStage : 0;
    // Shared memory outside the rings: alignment slack, barriers, epilogue patches, the position tables.  How many
    // tables the launch needs is known once every problem is planned: planned with four first, with kMaxTabs if that
    // was too few.
    for (int tabs_try = 4; tabs_try <= kMaxTabs; tabs_try += kMaxTabs - 4) {
        const int fixed = 1024 + 512 + kEpiWarps * kPatchBytes + tabs_try * kMaxPx * 8;
        bool seen[kMaxProb] = {};
        n_geo = acc_max = 0;
        for (int i0 = 0; i0 < n; ++i0) {
            if (seen[i0]) continue;
            // the set of this convolution: same level, same class
            int set[kMaxProb], m = 0;
            bool set_res = false;
            for (int j = i0; j < n; ++j)
                if (!seen[j] && level[j] == level[i0] && cls[j] == cls[i0]) set[m++] = j, seen[j] = true, set_res = set_res || ds[j]->residual_dev;
            // The staging area of residual operands is the top end of the ring area.  A set of 3x3 convolutions none of
            // which has a residual operand may lay its rings over it (the kernel then lets the epilogues that use the
            // area finish first); every other set stays below it.
            const bool under = resid && (set_res || ps[i0]->ksize != 3);
            // every problem is planned on its own first; where they disagree on the taps per weight stage, all are
            // planned again with the smallest (a stage per tap fits whatever fits three)
            int force_G = 0, a_max = 0, b_bytes = 0;
            for (int pass = 0; pass < 2; ++pass) {
                bool agree = true;
                int g_min = 9;
                a_max = 0;
                for (int q = 0; q < m; ++q) {
                    const int i = set[q];
                    rtoss_conv_desc dd = *ds[i];
                    static const int dummy = 0;
                    dd.residual_dev = under ? &dummy : nullptr;   // (only the plan's memory budget looks at it here)
                    int e = build_problem(ctx, ps[i], xs[i], ys[i], &dd, m, sms, &args[i], &pp[i], &mapA[i], &mapB[i], force_G, tabs_try);
                    if (e == (int)cudaErrorInvalidConfiguration) return -1;
                    if (e) return e;
                    args[i].resid = ds[i]->residual_dev;
                    args[i].resid_post = (ds[i]->residual_dev && ds[i]->residual_after_act) ? 1 : 0;
                    if (q == 0) b_bytes = pp[i].b_stage_bytes;
                    if (pp[i].b_stage_bytes != b_bytes || args[i].G != args[set[0]].G) agree = false;
                    if (args[i].G < g_min) g_min = args[i].G;
                    if (pp[i].a_stage_bytes > a_max) a_max = pp[i].a_stage_bytes;
                    if (pp[i].acc_cols > acc_max) acc_max = pp[i].acc_cols;
                    n_tiles[i] = (long)args[i].N * args[i].tiles_y * args[i].tiles_x * args[i].co_tiles;
                }
                if (agree) break;
                if (pass == 1) return -1;
                force_G = g_min;
            }
            // the rings every problem of the set fits into
            const int room = cap - fixed - (under ? res_bytes : 0);
            int na = (room - 2 * b_bytes) / a_max;
            if (na > kMaxA) na = kMaxA;
            bool one_block = true;   // (see plan_tc: layers of one channel block per tile keep more activation stages)
            for (int q = 0; q < m; ++q) one_block = one_block && ncb_of(ps[set[q]]) == 1;
            if (na > 2 && ps[i0]->ksize == 3 && !one_block) na = 2;
            if (na < 1) return -1;
            int nb = (room - na * a_max) / b_bytes;
            if (nb > kMaxB) nb = kMaxB;
            if (nb < 2) return -1;
            int gi = 0;
            while (gi < n_geo && !(geos[gi].a == a_max && geos[gi].b == b_bytes && geos[gi].na == na && geos[gi].nb == nb && geos[gi].under == under)) ++gi;
            if (gi == n_geo) geos[n_geo++] = Geo{a_max, b_bytes, na, nb, under};
            for (int q = 0; q < m; ++q) geo_of[set[q]] = gi;
        }
        // distinct position tables
        int n_distinct = 0;
        for (int i = 0; i < n; ++i) {
            bool fresh = true;
            for (int j = 0; j < i && fresh; ++j)
                fresh = !(args[j].Wq == args[i].Wq && args[j].TH == args[i].TH && args[j].TW == args[i].TW && args[j].N_px == args[i].N_px &&
                          args[j].Wo == args[i].Wo && args[j].y_c_stride == args[i].y_c_stride);
            n_distinct += fresh ? 1 : 0;
        }
        n_tabs_planned = tabs_try;
        if (n_distinct <= tabs_try) break;
        if (tabs_try == kMaxTabs) return -1;
    }
    const int fixed = 1024 + 512 + kEpiWarps * kPatchBytes + n_tabs_planned * kMaxPx * 8;
    // the launch's order: by level, inside a level by ring layout, then by falling tile count (stable)
    int order[kMaxProb];
    for (int i = 0; i < n; ++i) order[i] = i;
    for (int i = 1; i < n; ++i)
        for (int j = i; j > 0; --j) {
            const int u = order[j], v = order[j - 1];
            const bool before = level[u] != level[v] ? level[u] < level[v] : geo_of[u] != geo_of[v] ? geo_of[u] < geo_of[v] : n_tiles[u] > n_tiles[v];
            if (!before) break;
            std::swap(order[j], order[j - 1]);
        }
    int where[kMaxProb];   // position of convolution i in the launch
    for (int k = 0; k < n; ++k) where[order[k]] = k;
    g.n_prob = n;
    g.n_tabs = 0;
    g.ring_bytes = res_bytes;
    g.max_na = g.max_nb = 1;
    long units = 0;
    for (int k = 0; k < n; ++k) {
        const int i = order[k];
        TcArgs& a = g.prob[k];
        a = args[i];
        g.tmA[k] = mapA[i];
        g.tmB[k] = mapB[i];
        const Geo& ge = geos[geo_of[i]];
        a.NA = ge.na;
        a.NB = ge.nb;
        a.a_stage = (unsigned)ge.a;
        a.b_stage = (unsigned)ge.b;
        a.sB_off = (unsigned)ge.na * (unsigned)ge.a;
        a.geo = geo_of[i];
        const int ring = ge.na * ge.a + ge.nb * ge.b + (ge.under ? res_bytes : 0);
        if (ring > g.ring_bytes) g.ring_bytes = ring;
        if (ge.na > g.max_na) g.max_na = ge.na;
        if (ge.nb > g.max_nb) g.max_nb = ge.nb;
        // position table: shared with an earlier problem of the same tile geometry and output pitch
        a.tab = -1;
        for (int q = 0; q < k && a.tab < 0; ++q) {
            const TcArgs& b = g.prob[q];
            if (b.Wq == a.Wq && b.TH == a.TH && b.TW == a.TW && b.N_px == a.N_px && b.Wo == a.Wo && b.y_c_stride == a.y_c_stride) a.tab = b.tab;
        }
        if (a.tab < 0) {
            if (g.n_tabs == n_tabs_planned) return -1;
            a.tab = g.n_tabs++;
        }
        a.dep_mask = 0;
        if (after)
            for (int j = 0; j < i; ++j)
                if ((after[i] >> j) & 1u) a.dep_mask |= 1u << where[j];
        units += n_tiles[i];
        if (units > 0x3FFFFFFF) return -1;
        g.unit_end[k] = (int)units;
    }
    const int grid_n = (int)(units < sms ? units : sms);
    g.res_off = g.ring_bytes - res_bytes;
    for (int k = 0; k < n; ++k) {
        const long mine = n_tiles[order[k]];
        TcArgs& a = g.prob[k];
        a.done_target = (unsigned)((mine < grid_n ? mine : grid_n) * kEpiWarps);
        a.over_res = (resid && (int)(a.sB_off + (unsigned)a.NB * a.b_stage) > g.res_off) ? 1 : 0;
    }
    g.done = nullptr;
    if (chained) {
        // a block of counters of the context, taken in turn (launches that share a block must follow one another in a stream)
        g.done = ctx->chain_done + (size_t)(ctx->chain_next % RTOSS_CHAIN_SLOTS) * RTOSS_CHAIN_SLOT_WORDS;
        ctx->chain_next = (ctx->chain_next + 1) % RTOSS_CHAIN_SLOTS;
    }
    g.acc_stride = acc_max;
    launch_common(ctx, &g);
    if (g.tmem_cols > 512) return -1;
    const size_t smem_need = (size_t)fixed + (size_t)g.ring_bytes;
    if (smem_need > (size_t)cap) return -1;
    const size_t smem = smem_need > 116 * 1024 ? smem_need : 116 * 1024;
    dim3 grid((unsigned)grid_n);
    int e = ensure_smem_attr(ctx);
    if (e) return e;
    const bool bf = ps[0]->dtype == RTOSS_BF16, f32 = ps[0]->dtype == RTOSS_F32;
    cudaError_t le = f32 ? rtoss_dev::launch_pdl(conv_tc_kernel<float, TcLaunchN>, grid, kTcThreads, smem, (cudaStream_t)stream, 1, g)
                     : bf ? rtoss_dev::launch_pdl(conv_tc_kernel<__nv_bfloat16, TcLaunchN>, grid, kTcThreads, smem, (cudaStream_t)stream, 1, g)
                          : rtoss_dev::launch_pdl(conv_tc_kernel<__half, TcLaunchN>, grid, kTcThreads, smem, (cudaStream_t)stream, 1, g);
    return (int)le;
}

// Several independent convolutions of one class (kernel size, stride class, data type) in one launch.
int rtoss_launch_conv_tc_group(const rtoss_ctx* ctx, int n, const rtoss_packed* const* ps, const void* const* xs, void* const* ys,
                               const rtoss_conv_desc* const* ds, void* stream) {
    for (int i = 1; i < n; ++i) {
        if (ps[i]->ksize != ps[0]->ksize) return -1;
        if (ps[i]->ksize == 3 && ds[i]->stride != ds[0]->stride) return -1;   // (3x3: stride 2 stages four sub-tiles per block)
    }
    return rtoss_launch_conv_tc_chain(ctx, n, ps, xs, ys, ds, nullptr, stream);
}

int rtoss_tc_max_problems() { return kMaxProb; }
