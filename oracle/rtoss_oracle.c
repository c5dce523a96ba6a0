/*
 * R-TOSS CPU oracle  --  TEST INFRASTRUCTURE, NOT A PRODUCT PATH.
 *
 * A plain, slow, obviously-correct restatement of what the R-TOSS hot path
 * computes (arXiv 2303.02191): pattern table construction (Section IV.B,
 * Eq. 1 and criterion 1), per-kernel pattern selection (Section IV.C,
 * Algorithm 2; and a block-shared variant of it), the 1x1 -> 3x3 regrouping (Section IV.D, Algorithm 3), mask
 * application (Section II.B, "semi-structured pruning"), a canonical packed
 * form of the pruned weights (Section IV.C, last sentence), the layer
 * grouping (Section IV.A, Algorithm 1) and the inference convolution over
 * the pruned weights (Section II.B cost model).  Only tests, the smoke check
 * and the benchmark's cpu_baseline / reference legs may call it.  It shares
 * no code with the CUDA library and neither includes the other's headers.
 *
 * Parity pins: every function below is pinned by tests that do not call it
 * to produce their expectation (closed-form counts, brute force over all
 * C(9,k) subsets, top-k by sorting, library float64 convolution, unit
 * impulses, symmetries).  Exceptions, marked "parity unpinned" where they
 * stand: the CENTRE8 member list (the paper's pattern figure is not
 * available), and the details of the layer-grouping rule beyond the
 * invariants the paper states.
 *
 * Build: gcc -O2 -std=c11 -fopenmp -ffp-contract=off -fPIC -shared.
 * -ffp-contract=off matters: the selection arithmetic is defined with a
 * separately rounded multiply and separately rounded adds.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

/* ---- tap numbering: t = 3*r + c, r = row, c = column, bit t of a mask ---- */

static int popcount9(unsigned m) {
    int n = 0;
    for (int t = 0; t < 9; ++t) n += (m >> t) & 1u;
    return n;
}

/* Are the taps of mask m one 4-connected component?  (Section IV.B,
 * criterion 1, read as: the kept taps must hang together through
 * edge-adjacent neighbours.)  Flood fill from the lowest tap. */
static int connected4(unsigned m) {
    if (m == 0) return 0;
    unsigned seen = m & (~m + 1u); /* lowest set bit */
    for (;;) {
        unsigned grow = seen;
        for (int t = 0; t < 9; ++t) {
            if (!((seen >> t) & 1u)) continue;
            int r = t / 3, c = t % 3;
            if (r > 0) grow |= 1u << (t - 3);
            if (r < 2) grow |= 1u << (t + 3);
            if (c > 0) grow |= 1u << (t - 1);
            if (c < 2) grow |= 1u << (t + 1);
        }
        grow &= m;
        if (grow == seen) break;
        seen = grow;
    }
    return seen == m;
}

enum { PRESET_ALL = 0, PRESET_CONN4 = 1, PRESET_CENTRE8 = 2, PRESET_DENSE = 3 };

/*
 * Pattern presets.  Returns the number of masks written (ascending mask
 * order), or -1 on a bad argument / too small a capacity.
 *   ALL(k)    every k-subset of the 9 taps            (Eq. 1: C(9,k) of them)
 *   CONN4(k)  those forming one 4-connected component (criterion 1)
 *   CENTRE8   k = 4: connected 4-sets that contain the centre tap and are
 *             either a 2x2 block or the centre plus three of its four edge
 *             neighbours ("T" shapes).  parity unpinned: the paper's own
 *             pattern figure is not available, this is the 8-pattern set the
 *             small test configuration names.
 *   DENSE     the single mask with all 9 taps (k = 9)
 */
int oracle_pattern_preset(int k, int preset, uint16_t *masks, int capacity) {
    int n = 0;
    if (preset == PRESET_DENSE) {
        if (k != 9 || capacity < 1) return -1;
        masks[0] = 0x1FF;
        return 1;
    }
    if (k < 1 || k > 9) return -1;
    if (preset == PRESET_CENTRE8 && k != 4) return -1;
    for (unsigned m = 1; m < 512; ++m) {
        if (popcount9(m) != k) continue;
        int keep;
        if (preset == PRESET_ALL) {
            keep = 1;
        } else if (preset == PRESET_CONN4) {
            keep = connected4(m);
        } else if (preset == PRESET_CENTRE8) {
            keep = 0;
            if ((m >> 4) & 1u) {
                /* 2x2 block: rows {r0,r0+1}, columns {c0,c0+1} */
                for (int r0 = 0; r0 < 2; ++r0)
                    for (int c0 = 0; c0 < 2; ++c0) {
                        unsigned b = (1u << (3 * r0 + c0)) | (1u << (3 * r0 + c0 + 1)) |
                                     (1u << (3 * r0 + 3 + c0)) | (1u << (3 * r0 + 3 + c0 + 1));
                        if (b == m) keep = 1;
                    }
                /* T shape: centre + three of the edge neighbours 1,3,5,7 */
                unsigned edges = (1u << 1) | (1u << 3) | (1u << 5) | (1u << 7);
                unsigned rest = m & ~(1u << 4);
                if ((rest & ~edges) == 0 && popcount9(rest) == 3) keep = 1;
            }
        } else {
            return -1;
        }
        if (keep) {
            if (n >= capacity) return -1;
            masks[n++] = (uint16_t)m;
        }
    }
    return n;
}

/* A table is valid when every mask is in 1..511 with exactly k taps and no
 * mask appears twice.  Returns 1 / 0. */
int oracle_pattern_table_valid(const uint16_t *masks, int P, int k) {
    if (P < 1 || P > 255 || k < 1 || k > 9) return 0;
    for (int p = 0; p < P; ++p) {
        if (masks[p] == 0 || masks[p] > 511 || popcount9(masks[p]) != k) return 0;
        for (int q = 0; q < p; ++q)
            if (masks[q] == masks[p]) return 0;
    }
    return 1;
}

/* ---- selection (Algorithm 2) ------------------------------------------- */

/*
 * For each of n 3x3 kernels (9 consecutive floats, row-major taps) find the
 * pattern that retains the largest L2 norm.  The norm of the kernel under a
 * pattern is compared through its square: S_p = sum over the pattern's taps
 * of w_t^2.  Arithmetic is fixed so that the integer result is reproducible:
 * q_t = w_t*w_t rounded to float; S_p accumulated in float over the taps in
 * ascending order starting from 0; the first pattern with a strictly larger
 * sum wins (so ties go to the lowest pattern id, and a NaN sum never wins).
 */
void oracle_select_kernels(const float *w, long n, const uint16_t *masks, int P, uint8_t *pid) {
#pragma omp parallel for schedule(static)
    for (long i = 0; i < n; ++i) {
        const float *kw = w + 9 * i;
        float q[9];
        for (int t = 0; t < 9; ++t) {
            volatile float sq = kw[t] * kw[t];
            q[t] = sq;
        }
        int best = 0;
        float best_s = 0.0f;
        for (int p = 0; p < P; ++p) {
            volatile float s = 0.0f;
            for (int t = 0; t < 9; ++t)
                if ((masks[p] >> t) & 1u) s = s + q[t];
            float sv = s;
            if (p == 0) {
                best_s = sv;
            } else if (sv > best_s || (best_s != best_s && sv == sv)) {
                /* strictly larger, or the running best is NaN and this is not */
                best = p;
                best_s = sv;
            }
        }
        pid[i] = (uint8_t)best;
    }
}

/* 3x3 layer: weights [Cout][Cin][3][3]; one pattern id per (co, ci). */
void oracle_select_3x3(const float *w, int Cout, int Cin, const uint16_t *masks, int P, uint8_t *pid) {
    oracle_select_kernels(w, (long)Cout * Cin, masks, P, pid);
}

/*
 * 1x1 layer (Algorithm 3): flatten the [Cout][Cin] weights filter-major,
 * cut the list into runs of 9, view each full run as a row-major 3x3
 * matrix, and run the 3x3 selection on those temporaries.  Returns the
 * number of full runs G = floor(Cout*Cin/9); pid1 has G entries.  The
 * Cout*Cin - 9G left-over weights at the end of the list are pruned.
 */
long oracle_select_1x1(const float *w, int Cout, int Cin, const uint16_t *masks, int P, uint8_t *pid1) {
    /* w is [Cout][Cin] contiguous, so the filter-major flat list is w itself: weight e = co*Cin + ci.
     * Run g is w[9g .. 9g+8], already in the order of a row-major 3x3; only full runs are selected on. */
    const long G = ((long)Cout * Cin) / 9;
    oracle_select_kernels(w, G, masks, P, pid1);
    return G;
}

/* ---- selection with one pattern per block of kernels (a variant, not the paper's per-kernel rule) ---- */

/*
 * Section IV.C lets the kernels of a layer group take over one kernel mask; this variant applies that idea
 * inside a layer: the kernels (co, ci) with co in a block of FB consecutive filters and ci in a block of CB
 * consecutive input channels all get ONE pattern, the one that retains the most energy of the whole block.
 * (It changes which weights survive, so it is a different pruning result from Algorithm 2; it exists because a
 * pattern shared by a block lets a matrix unit skip the pruned taps of the whole block.)
 *
 *   q[co][ci][t]  = w*w rounded to float (as in Algorithm 2's restatement above), then widened to double
 *   r[co][t]      = sum over the block's channels ci, ascending, in double
 *   E[t]          = sum over the block's filters co, ascending, of r[co][t], in double
 *   S_p           = sum over the taps t of mask p, ascending, of E[t], in double
 *   pattern       = first p with a strictly larger S_p (ties -> lowest id; a NaN sum never wins)
 *
 * FB = CB = 1 is Algorithm 2 with double instead of float pattern sums.  Blocks at the ragged end of the
 * filter or channel range are simply smaller.  pid gets Cout*Cin entries, constant inside a block.
 */
void oracle_select_shared(const float *w, int Cout, int Cin, int FB, int CB, const uint16_t *masks, int P, uint8_t *pid) {
    for (int co0 = 0; co0 < Cout; co0 += FB)
        for (int ci0 = 0; ci0 < Cin; ci0 += CB) {
            int co1 = co0 + FB < Cout ? co0 + FB : Cout;
            int ci1 = ci0 + CB < Cin ? ci0 + CB : Cin;
            double E[9];
            for (int t = 0; t < 9; ++t) E[t] = 0.0;
            for (int co = co0; co < co1; ++co) {
                double r[9];
                for (int t = 0; t < 9; ++t) r[t] = 0.0;
                for (int ci = ci0; ci < ci1; ++ci) {
                    const float *kw = w + 9 * ((long)co * Cin + ci);
                    for (int t = 0; t < 9; ++t) {
                        volatile float sq = kw[t] * kw[t];
                        r[t] = r[t] + (double)sq;
                    }
                }
                for (int t = 0; t < 9; ++t) E[t] = E[t] + r[t];
            }
            int best = 0;
            double best_s = 0.0;
            for (int p = 0; p < P; ++p) {
                double sv = 0.0;
                for (int t = 0; t < 9; ++t)
                    if ((masks[p] >> t) & 1u) sv = sv + E[t];
                if (p == 0) {
                    best_s = sv;
                } else if (sv > best_s || (best_s != best_s && sv == sv)) {
                    best = p;
                    best_s = sv;
                }
            }
            for (int co = co0; co < co1; ++co)
                for (int ci = ci0; ci < ci1; ++ci) pid[(long)co * Cin + ci] = (uint8_t)best;
        }
}

/* ---- mask application ---------------------------------------------------- */

/* W <- W (.) mask(pid): weights outside the chosen pattern become +0. */
void oracle_mask_3x3(const float *w, int Cout, int Cin, const uint16_t *masks, const uint8_t *pid, float *wm) {
    long n = (long)Cout * Cin;
    for (long i = 0; i < n; ++i)
        for (int t = 0; t < 9; ++t) wm[9 * i + t] = ((masks[pid[i]] >> t) & 1u) ? w[9 * i + t] : 0.0f;
}

/* 1x1: position e of the flat list belongs to run g = e/9 at tap e%9; runs
 * beyond the last full one are zeroed. */
void oracle_mask_1x1(const float *w, int Cout, int Cin, const uint16_t *masks, const uint8_t *pid1, float *wm) {
    long len = (long)Cout * Cin, G = len / 9;
    for (long e = 0; e < len; ++e) {
        long g = e / 9;
        int t = (int)(e % 9);
        wm[e] = (g < G && ((masks[pid1[g]] >> t) & 1u)) ? w[e] : 0.0f;
    }
}

/* ---- rounding to the storage types -------------------------------------- */

static uint32_t f2u(float f) { uint32_t u; memcpy(&u, &f, 4); return u; }
static float u2f(uint32_t u) { float f; memcpy(&f, &u, 4); return f; }

/* float -> bfloat16 bits, round to nearest even; NaN stays a quiet NaN. */
uint16_t oracle_f32_to_bf16_bits(float f) {
    uint32_t u = f2u(f);
    if ((u & 0x7F800000u) == 0x7F800000u && (u & 0x007FFFFFu)) return (uint16_t)((u >> 16) | 0x0040u);
    uint32_t lsb = (u >> 16) & 1u;
    u += 0x7FFFu + lsb;
    return (uint16_t)(u >> 16);
}
float oracle_bf16_bits_to_f32(uint16_t h) { return u2f((uint32_t)h << 16); }

/* float -> IEEE binary16 bits, round to nearest even, with subnormals and
 * overflow to infinity. */
uint16_t oracle_f32_to_f16_bits(float f) {
    uint32_t u = f2u(f);
    uint32_t sign = (u >> 16) & 0x8000u;
    uint32_t absu = u & 0x7FFFFFFFu;
    if (absu >= 0x7F800000u) return (uint16_t)(sign | (absu > 0x7F800000u ? 0x7E00u : 0x7C00u));
    double a = fabs((double)f);
    if (a == 0.0) return (uint16_t)sign;
    int e;
    double m = frexp(a, &e); /* a = m * 2^e, m in [0.5,1) */
    /* binary16: normal numbers 2^-14 .. 65504, spacing 2^(E-10); subnormal spacing 2^-24 */
    int E = e - 1; /* a = (2m) * 2^E, 2m in [1,2) */
    (void)m;
    double quantum = (E < -14) ? ldexp(1.0, -24) : ldexp(1.0, E - 10);
    double q = a / quantum; /* exact: power-of-two scaling */
    double fl = floor(q);
    double rem = q - fl;
    if (rem > 0.5 || (rem == 0.5 && fmod(fl, 2.0) == 1.0)) fl += 1.0;
    double r = fl * quantum; /* rounded magnitude */
    if (r > 65504.0) return (uint16_t)(sign | 0x7C00u);
    if (r < ldexp(1.0, -14)) return (uint16_t)(sign | (uint32_t)(r / ldexp(1.0, -24)));
    int e2;
    double m2 = frexp(r, &e2); /* r = m2 * 2^e2 */
    int E2 = e2 - 1;
    uint32_t mant = (uint32_t)((m2 * 2.0 - 1.0) * 1024.0);
    return (uint16_t)(sign | ((uint32_t)(E2 + 15) << 10) | mant);
}
float oracle_f16_bits_to_f32(uint16_t h) {
    uint32_t sign = (h >> 15) & 1u, ex = (h >> 10) & 0x1Fu, mant = h & 0x3FFu;
    double v;
    if (ex == 0x1F) v = mant ? NAN : INFINITY;
    else if (ex == 0) v = ldexp((double)mant, -24);
    else v = ldexp(1.0 + (double)mant / 1024.0, (int)ex - 15);
    return (float)(sign ? -v : v);
}

enum { DT_F32 = 0, DT_BF16 = 1, DT_F16 = 2 };

/* Round a float to the given storage type and return it as a float. */
float oracle_round_to(float v, int dtype) {
    if (dtype == DT_BF16) return oracle_bf16_bits_to_f32(oracle_f32_to_bf16_bits(v));
    if (dtype == DT_F16) return oracle_f16_bits_to_f32(oracle_f32_to_f16_bits(v));
    return v;
}
void oracle_round_array(const float *in, long n, int dtype, float *out) {
    for (long i = 0; i < n; ++i) out[i] = oracle_round_to(in[i], dtype);
}

/* ---- canonical packed form ---------------------------------------------- */

/*
 * 3x3 pack.  val[(co*Cin+ci)*k + j] is the weight at the j-th kept tap
 * (ascending tap index) of kernel (co,ci), rounded to the compute type and
 * returned as float.  "Kernels with similar patterns are grouped together"
 * (Section IV.C) is given this concrete form: for every input channel ci a
 * stable counting sort of the filters by pattern id,
 *   perm[ci*Cout + i]          = filter at position i (pid ascending, then co)
 *   bucket_off[ci*(P+1) + p]   = first position of pattern p; entry P = Cout.
 */
void oracle_pack_3x3(const float *w, int Cout, int Cin, const uint16_t *masks, int P, int k,
                     const uint8_t *pid, int compute_dtype, float *val, uint32_t *perm, uint32_t *bucket_off) {
    for (long i = 0; i < (long)Cout * Cin; ++i) {
        int j = 0;
        for (int t = 0; t < 9; ++t)
            if ((masks[pid[i]] >> t) & 1u) val[i * k + j++] = oracle_round_to(w[9 * i + t], compute_dtype);
    }
    for (int ci = 0; ci < Cin; ++ci) {
        uint32_t pos = 0;
        for (int p = 0; p < P; ++p) {
            bucket_off[(long)ci * (P + 1) + p] = pos;
            for (int co = 0; co < Cout; ++co)
                if (pid[(long)co * Cin + ci] == p) perm[(long)ci * Cout + pos++] = (uint32_t)co;
        }
        bucket_off[(long)ci * (P + 1) + P] = pos;
    }
}

/* 1x1 pack: val1[g*k + j] for the G full runs, natural order, no reorder. */
void oracle_pack_1x1(const float *w, int Cout, int Cin, const uint16_t *masks, int k, const uint8_t *pid1,
                     int compute_dtype, float *val1) {
    long G = ((long)Cout * Cin) / 9;
    for (long g = 0; g < G; ++g) {
        int j = 0;
        for (int t = 0; t < 9; ++t)
            if ((masks[pid1[g]] >> t) & 1u) val1[g * k + j++] = oracle_round_to(w[9 * g + t], compute_dtype);
    }
}

/* Packed -> dense masked weights (the inverse view of the two packs). */
void oracle_unpack_3x3(const float *val, int Cout, int Cin, const uint16_t *masks, int k, const uint8_t *pid, float *wd) {
    for (long i = 0; i < (long)Cout * Cin; ++i) {
        int j = 0;
        for (int t = 0; t < 9; ++t) wd[9 * i + t] = ((masks[pid[i]] >> t) & 1u) ? val[i * k + j++] : 0.0f;
    }
}
void oracle_unpack_1x1(const float *val1, int Cout, int Cin, const uint16_t *masks, int k, const uint8_t *pid1, float *wd) {
    long len = (long)Cout * Cin, G = len / 9;
    for (long e = 0; e < len; ++e) wd[e] = 0.0f;
    for (long g = 0; g < G; ++g) {
        int j = 0;
        for (int t = 0; t < 9; ++t)
            if ((masks[pid1[g]] >> t) & 1u) wd[9 * g + t] = val1[g * k + j++];
    }
}

/* ---- convolution over the pruned (dense masked) weights ----------------- */

enum { ACT_NONE = 0, ACT_RELU = 1, ACT_SILU = 2 };

static double activate(double v, int act) {
    if (act == ACT_RELU) return v > 0.0 ? v : 0.0;
    if (act == ACT_SILU) return v / (1.0 + exp(-v));
    return v;
}

/* One output element of the 3x3 convolution (cross-correlation, zero
 * padding 1): sum over ci, r, c in that order in double, then bias,
 * activation, one rounding to the output type. */
static float conv3x3_at(const float *x, int Cin, int H, int W, const float *wd, const float *bias, int stride,
                        int act, int out_dtype, int n, int co, int oy, int ox) {
    double acc = 0.0;
    for (int ci = 0; ci < Cin; ++ci)
        for (int r = 0; r < 3; ++r)
            for (int c = 0; c < 3; ++c) {
                int iy = oy * stride + r - 1, ix = ox * stride + c - 1;
                if (iy < 0 || iy >= H || ix < 0 || ix >= W) continue;
                acc += (double)wd[((long)co * Cin + ci) * 9 + 3 * r + c] *
                       (double)x[(((long)n * Cin + ci) * H + iy) * W + ix];
            }
    if (bias) acc += (double)bias[co];
    return oracle_round_to((float)activate(acc, act), out_dtype);
}

/* x [N][Cin][H][W], wd [Cout][Cin][3][3] (already masked and rounded),
 * y [N][Cout][Ho][Wo], Ho = (H+2-3)/stride+1. */
void oracle_conv3x3(const float *x, int N, int Cin, int H, int W, const float *wd, int Cout, const float *bias,
                    int stride, int act, int out_dtype, float *y) {
    int Ho = (H - 1) / stride + 1, Wo = (W - 1) / stride + 1;
#pragma omp parallel for collapse(2) schedule(static)
    for (int n = 0; n < N; ++n)
        for (int co = 0; co < Cout; ++co)
            for (int oy = 0; oy < Ho; ++oy)
                for (int ox = 0; ox < Wo; ++ox)
                    y[(((long)n * Cout + co) * Ho + oy) * Wo + ox] =
                        conv3x3_at(x, Cin, H, W, wd, bias, stride, act, out_dtype, n, co, oy, ox);
}

/* Selected output elements only: idx holds (n, co, oy, ox) quadruples. */
void oracle_conv3x3_points(const float *x, int N, int Cin, int H, int W, const float *wd, int Cout,
                           const float *bias, int stride, int act, int out_dtype, const int *idx, long npts,
                           float *out) {
    (void)N; (void)Cout;
#pragma omp parallel for schedule(static)
    for (long i = 0; i < npts; ++i)
        out[i] = conv3x3_at(x, Cin, H, W, wd, bias, stride, act, out_dtype, idx[4 * i], idx[4 * i + 1],
                            idx[4 * i + 2], idx[4 * i + 3]);
}

static float conv1x1_at(const float *x, int Cin, int H, int W, const float *wd, const float *bias, int stride,
                        int act, int out_dtype, int n, int co, int oy, int ox) {
    double acc = 0.0;
    for (int ci = 0; ci < Cin; ++ci)
        acc += (double)wd[(long)co * Cin + ci] * (double)x[(((long)n * Cin + ci) * H + oy * stride) * W + ox * stride];
    if (bias) acc += (double)bias[co];
    return oracle_round_to((float)activate(acc, act), out_dtype);
}

/* 1x1, no padding: Ho = (H-1)/stride+1. wd [Cout][Cin] masked and rounded. */
void oracle_conv1x1(const float *x, int N, int Cin, int H, int W, const float *wd, int Cout, const float *bias,
                    int stride, int act, int out_dtype, float *y) {
    int Ho = (H - 1) / stride + 1, Wo = (W - 1) / stride + 1;
#pragma omp parallel for collapse(2) schedule(static)
    for (int n = 0; n < N; ++n)
        for (int co = 0; co < Cout; ++co)
            for (int oy = 0; oy < Ho; ++oy)
                for (int ox = 0; ox < Wo; ++ox)
                    y[(((long)n * Cout + co) * Ho + oy) * Wo + ox] =
                        conv1x1_at(x, Cin, H, W, wd, bias, stride, act, out_dtype, n, co, oy, ox);
}

void oracle_conv1x1_points(const float *x, int N, int Cin, int H, int W, const float *wd, int Cout,
                           const float *bias, int stride, int act, int out_dtype, const int *idx, long npts,
                           float *out) {
    (void)N; (void)Cout;
#pragma omp parallel for schedule(static)
    for (long i = 0; i < npts; ++i)
        out[i] = conv1x1_at(x, Cin, H, W, wd, bias, stride, act, out_dtype, idx[4 * i], idx[4 * i + 1],
                            idx[4 * i + 2], idx[4 * i + 3]);
}

/* ---- layer grouping (Algorithm 1) ---------------------------------------- */

/*
 * The model is an explicit DAG of nodes in topological order.  Node i has
 * kind[i] (1 = convolution layer, 0 = any other operation), and for
 * convolutions cout/cin/ksize; its inputs are in_idx[in_off[i] ..
 * in_off[i+1]).  For every convolution l, a depth-first search walks
 * backwards from l's inputs (in listed order, through non-convolution nodes)
 * and the first convolution reached is its parent: one parent per child, many
 * children per parent.  A layer with no convolution upstream is its own
 * parent and founds a group.  A child joins its parent's group when it has
 * the parent's kernel size and (Cout, Cin) -- only then can the parent's
 * per-kernel patterns be shared index by index -- otherwise it founds a new
 * group.  parent[i] = -1 and group[i] = -1 for non-convolution nodes.
 * parity unpinned beyond: one parent per layer, roots are their own parents,
 * groups partition the convolutions, members of a group have equal shapes.
 * Returns the number of groups.
 */
static int dfs_first_conv(int node, const int *kind, const int *in_off, const int *in_idx) {
    for (int e = in_off[node]; e < in_off[node + 1]; ++e) {
        int u = in_idx[e];
        if (kind[u] == 1) return u;
        int f = dfs_first_conv(u, kind, in_off, in_idx);
        if (f >= 0) return f;
    }
    return -1;
}

int oracle_group_layers(int L, const int *kind, const int *cout, const int *cin, const int *ksize,
                        const int *in_off, const int *in_idx, int *parent, int *group) {
    int ngroups = 0;
    for (int l = 0; l < L; ++l) {
        parent[l] = -1;
        group[l] = -1;
        if (kind[l] != 1) continue;
        int p = dfs_first_conv(l, kind, in_off, in_idx);
        if (p < 0) {
            parent[l] = l;
            group[l] = ngroups++;
        } else {
            parent[l] = p;
            if (ksize[p] == ksize[l] && cout[p] == cout[l] && cin[p] == cin[l]) group[l] = group[p];
            else group[l] = ngroups++;
        }
    }
    return ngroups;
}

/* ---- glue operations of a whole network (outside the paper's method; NCHW) ---- */

/* k x k max-pooling with stride; padded positions are ignored (they count as minus infinity). */
void oracle_maxpool2d(const float *x, int N, int C, int H, int W, int k, int stride, int pad, float *y) {
    int Ho = (H + 2 * pad - k) / stride + 1, Wo = (W + 2 * pad - k) / stride + 1;
    for (long nc = 0; nc < (long)N * C; ++nc)
        for (int oh = 0; oh < Ho; ++oh)
            for (int ow = 0; ow < Wo; ++ow) {
                float m = -INFINITY;
                for (int dy = 0; dy < k; ++dy)
                    for (int dx = 0; dx < k; ++dx) {
                        int ih = oh * stride + dy - pad, iw = ow * stride + dx - pad;
                        if (ih < 0 || ih >= H || iw < 0 || iw >= W) continue;
                        float v = x[(nc * H + ih) * W + iw];
                        if (v > m) m = v;
                    }
                y[(nc * Ho + oh) * Wo + ow] = m;
            }
}

/* nearest-neighbour up-sampling by two */
void oracle_upsample2x(const float *x, int N, int C, int H, int W, float *y) {
    for (long nc = 0; nc < (long)N * C; ++nc)
        for (int oh = 0; oh < 2 * H; ++oh)
            for (int ow = 0; ow < 2 * W; ++ow) y[(nc * 2 * H + oh) * 2 * W + ow] = x[(nc * H + oh / 2) * W + ow / 2];
}

/* y = act(a + b), sum in double, one rounding to the storage type */
void oracle_add_act(const float *a, const float *b, long n, int act, int out_dtype, float *y) {
    for (long i = 0; i < n; ++i) y[i] = oracle_round_to((float)activate((double)a[i] + (double)b[i], act), out_dtype);
}
