/*
 * librtoss -- R-TOSS hot path on NVIDIA B200 (sm_100a), C ABI.
 *
 * R-TOSS (arXiv 2303.02191) prunes every 3x3 convolution kernel to the k taps
 * of one pattern out of a small pattern table, choosing per kernel the pattern
 * that retains the largest L2 norm (Section IV.C, Algorithm 2); 1x1 weights
 * are first regrouped, nine at a time, into temporary 3x3 matrices and pruned
 * with the same patterns (Section IV.D, Algorithm 3).  This library performs
 * that selection on the GPU, packs the surviving weights, and runs inference
 * convolution directly on the packed form.
 *
 * Conventions
 *   - Tap numbering inside a 3x3 kernel: t = 3*row + col.  A pattern is a
 *     9-bit mask, bit t set = tap t kept; every mask of a table has exactly k
 *     bits.  A pattern id ("pid") is an index into the table.
 *   - Pointers named *_dev are device pointers on the context's device,
 *     *_host are host pointers.  The caller owns every buffer it passes.
 *     Device pointers of tensors must be 16-byte aligned.
 *   - `cuda_stream` is a cudaStream_t passed as void* (NULL = default stream).
 *     Calls only enqueue work on it and never synchronise, unless stated.
 *   - Every call returns an rtoss_status; argument errors are detected on the
 *     host before anything is launched.  Nothing throws or aborts.
 *   - There is no CPU fallback: without a CUDA device rtoss_create fails.
 */
#ifndef RTOSS_H
#define RTOSS_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    RTOSS_OK = 0,
    RTOSS_ERR_INVALID_ARG = 1,       /* null pointer, non-positive size, bad enum */
    RTOSS_ERR_BAD_PATTERN_TABLE = 2, /* mask outside 1..511, popcount != k, duplicate, P outside 1..255 */
    RTOSS_ERR_UNSUPPORTED = 3,       /* valid request the library has no kernel for */
    RTOSS_ERR_ALIGNMENT = 4,         /* a tensor pointer is not 16-byte aligned */
    RTOSS_ERR_ALLOC = 5,             /* device or host allocation failed */
    RTOSS_ERR_CUDA = 6,              /* a CUDA runtime call failed; see rtoss_last_error */
    RTOSS_ERR_TIMEOUT = 7            /* a bounded device-side wait gave up */
} rtoss_status;

typedef enum { RTOSS_F32 = 0, RTOSS_BF16 = 1, RTOSS_F16 = 2 } rtoss_dtype;
typedef enum { RTOSS_NCHW = 0, RTOSS_NHWC = 1 } rtoss_layout;
typedef enum { RTOSS_ACT_NONE = 0, RTOSS_ACT_RELU = 1, RTOSS_ACT_SILU = 2 } rtoss_act;
typedef enum {
    RTOSS_PRESET_ALL = 0,     /* every k-subset of the 9 taps (Eq. 1) */
    RTOSS_PRESET_CONN4 = 1,   /* k-subsets forming one edge-connected set (Section IV.B, criterion 1) */
    RTOSS_PRESET_CENTRE8 = 2, /* k = 4: the four 2x2 blocks through the centre + the four T shapes */
    RTOSS_PRESET_DENSE = 3    /* k = 9: the single all-taps mask (no pruning) */
} rtoss_preset;

typedef enum {
    RTOSS_PATH_AUTO = 0,   /* tensor path where the call qualifies, FMA path otherwise */
    RTOSS_PATH_FMA = 1,    /* FP32 FMA pipes (any dtype, layout, stride); the pruned taps are multiplied as zeros */
    RTOSS_PATH_TENSOR = 2  /* masked dense implicit GEMM on tcgen05; RTOSS_ERR_UNSUPPORTED if the call does not qualify */
} rtoss_path;

typedef struct rtoss_ctx rtoss_ctx;       /* per-device state: error text, host-path workspace */
typedef struct rtoss_packed rtoss_packed; /* one layer's pruned weights in packed form, on the device */

/* Create / destroy a context on CUDA device `device`.  rtoss_create fails with
 * RTOSS_ERR_CUDA when the device cannot be used.  rtoss_destroy frees the
 * context's workspace; packed handles are freed separately. */
rtoss_status rtoss_create(int device, rtoss_ctx** ctx);
void rtoss_destroy(rtoss_ctx* ctx);
const char* rtoss_status_string(rtoss_status s);
/* Text of the last error recorded on this context ("" if none).  Valid until
 * the next failing call on the same context. */
const char* rtoss_last_error(const rtoss_ctx* ctx);

/* ---- host-only steps (no GPU needed) ------------------------------------- */

/* Pattern table presets (Section IV.B: Eq. 1 enumerates all C(9,k) masks;
 * criterion 1 drops those whose kept taps are not adjacent).  Writes the masks
 * in ascending numeric order into masks_host.  *P is the capacity on entry and
 * the count on return.  RTOSS_ERR_INVALID_ARG for a bad k/preset pairing or
 * too small a capacity. */
rtoss_status rtoss_pattern_preset(int k, rtoss_preset preset, uint16_t* masks_host, int* P);

/* Check a caller-supplied table: 1 <= P <= 255, 1 <= k <= 9, every mask in
 * 1..511 with exactly k bits, no duplicates.  RTOSS_OK or
 * RTOSS_ERR_BAD_PATTERN_TABLE. */
rtoss_status rtoss_pattern_table_validate(const uint16_t* masks_host, int P, int k);

/* One node of the model graph for the layer grouping.  Nodes are listed in
 * topological order; `inputs` holds the ids of the producing nodes. */
typedef struct {
    int is_conv;       /* 1 = convolution layer, 0 = any other operation */
    int cout, cin;     /* convolution shape (ignored for other nodes) */
    int ksize;         /* 1 or 3 (ignored for other nodes) */
    int n_inputs;
    const int* inputs; /* n_inputs node ids, each < this node's id */
} rtoss_layer_node;

/* Layer grouping by depth-first search (Section IV.A, Algorithm 1).  For each
 * convolution the search walks backwards from its inputs, in listed order and
 * through non-convolution nodes, and the first convolution reached is its
 * parent (one parent per child).  A convolution with none upstream is its own
 * parent and founds a group.  A child joins its parent's group when it has the
 * parent's kernel size and (cout, cin) -- then it may reuse the parent's
 * pattern ids kernel by kernel -- otherwise it founds a new group.
 * parent[i] = group[i] = -1 for non-convolution nodes.  *n_groups (nullable)
 * receives the group count.  RTOSS_ERR_INVALID_ARG on a malformed graph. */
rtoss_status rtoss_group_layers(const rtoss_layer_node* nodes, int L, int* parent, int* group, int* n_groups);

/* ---- selection (Algorithm 2; Algorithm 3 for ksize = 1) -------------------- */

/* For every kernel, the id of the pattern that retains the largest sum of
 * squared weights (equivalently the largest L2 norm).  The arithmetic is
 * fixed so that ids are reproducible bit for bit: squares rounded to fp32,
 * summed in fp32 over the pattern's taps in ascending order, first strictly
 * larger sum wins (ties -> lowest id; a NaN sum never wins).
 *   ksize = 3: w_dev is [Cout][Cin][3][3] contiguous; pid_dev gets Cout*Cin
 *              bytes, pid_dev[co*Cin+ci].
 *   ksize = 1: w_dev is [Cout][Cin]; the flat list is cut into G =
 *              floor(Cout*Cin/9) runs of nine, run g viewed as a row-major
 *              3x3; pid_dev gets G bytes.  The Cout*Cin - 9G trailing weights
 *              are pruned by the later steps.
 * w_dtype may be fp32, bf16 or fp16 (widened exactly).  masks_host is
 * validated (RTOSS_ERR_BAD_PATTERN_TABLE). */
rtoss_status rtoss_select_patterns(rtoss_ctx* ctx, const void* w_dev, rtoss_dtype w_dtype, int Cout, int Cin,
                                   int ksize, const uint16_t* masks_host, int P, int k, uint8_t* pid_dev,
                                   void* cuda_stream);

/* Pattern usage over a sample of kernels (Section IV.B, criterion 2: keep the most used patterns, judged by the
 * L2 norm on random kernels in [-1, 1]).  kernels_dev holds n_kernels 3x3 kernels (9 values each, the caller's
 * random sample); every kernel is matched against the candidate table exactly as rtoss_select_patterns does and
 * counts_dev[p] (P entries, uint64, zeroed by the call) receives how many kernels chose pattern p.  Ranking the
 * counts and cutting the table is left to the caller (ties: lower pattern id first).  pid_scratch_dev is a
 * caller-owned buffer of n_kernels bytes. */
rtoss_status rtoss_pattern_usage(rtoss_ctx* ctx, const void* kernels_dev, rtoss_dtype dtype, int64_t n_kernels,
                                 const uint16_t* masks_host, int P, int k, uint8_t* pid_scratch_dev, uint64_t* counts_dev,
                                 void* cuda_stream);

/* Criterion 2, the cut (Section IV.B: only the most frequently chosen patterns stay): rank the candidates of a table by
 * their usage counts -- most used first; equal counts: the numerically lower mask first -- and keep the best M.
 * order_host (P entries, may be NULL) receives the candidate indices in rank order; top_masks_host (M entries) the
 * kept masks in ascending numeric order, i.e. a table every other call accepts.  Host only.  How many to keep is
 * the caller's choice: the paper gives no cut-off.  RTOSS_ERR_BAD_PATTERN_TABLE for an invalid candidate table,
 * RTOSS_ERR_INVALID_ARG for null pointers or M outside 1..P. */
rtoss_status rtoss_pattern_rank(const uint16_t* masks_host, const uint64_t* counts_host, int P, int k, int M,
                                uint16_t* top_masks_host, int* order_host);

/* Pattern-set derivation in one call (Section IV.B): the candidates are the preset table for k (RTOSS_PRESET_ALL:
 * Eq. 1 alone; RTOSS_PRESET_CONN4: Eq. 1 and the adjacency criterion), their usage over the caller's sample of
 * kernels is counted on the GPU exactly as rtoss_pattern_usage does (same arguments: kernels_dev, pid_scratch_dev
 * of n_kernels bytes, counts_dev with room for 255 counters), the stream is synchronised, and the M most used are
 * returned as rtoss_pattern_rank returns them (M larger than the number of candidates keeps them all).
 * *P_candidates receives the number of candidates, *M_kept the number of masks written to top_masks_host (room for
 * M); cand_masks_host / cand_counts_host (room for 255 entries each, may be NULL) the candidate table and its
 * counts.  The random sample is the caller's (the paper asks for values in [-1, 1]; count and seed are not given). */
rtoss_status rtoss_pattern_table_derive(rtoss_ctx* ctx, const void* kernels_dev, rtoss_dtype dtype, int64_t n_kernels,
                                        int k, rtoss_preset preset, int M, uint8_t* pid_scratch_dev, uint64_t* counts_dev,
                                        uint16_t* top_masks_host, int* M_kept, uint16_t* cand_masks_host,
                                        uint64_t* cand_counts_host, int* P_candidates, void* cuda_stream);

/* A variant of the selection, not the paper's per-kernel rule: ONE pattern for every block of `filter_block`
 * consecutive filters x `channel_block` consecutive input channels of a 3x3 layer, namely the pattern that retains the
 * largest sum of squared weights of the whole block (Section IV.C shares kernel masks inside layer groups; this
 * shares them inside a layer).  pid_dev gets Cout*Cin ids as rtoss_select_patterns writes them, constant inside a
 * block, so rtoss_pack and the convolutions take them unchanged.  Why: with filter_block = 128 and channel_block a
 * multiple of 16 the tensor path multiplies only the k kept taps of every block (9/k fewer matrix instructions), which
 * per-kernel patterns never allow.  The price is retained norm: the result is a different (coarser) pruning than
 * Algorithm 2's, whose effect on detection accuracy this library cannot measure.
 * Arithmetic (fixed, so that ids are reproducible): squares rounded to fp32, then summed in double over the block's
 * channels (ascending) per filter, over the block's filters (ascending), over the pattern's taps (ascending); first
 * strictly larger sum wins.  Blocks at the ragged end of a range are smaller.  1 <= filter_block <= 256,
 * channel_block >= 1; ksize 3 only.  Errors as rtoss_select_patterns. */
rtoss_status rtoss_select_patterns_shared(rtoss_ctx* ctx, const void* w_dev, rtoss_dtype w_dtype, int Cout, int Cin,
                                          int filter_block, int channel_block, const uint16_t* masks_host, int P, int k,
                                          uint8_t* pid_dev, void* cuda_stream);

/* ---- packing (Section IV.C, last sentence: kernels of like pattern are put together) --- */

/* Build the packed form of one layer from its weights and pattern ids:
 *   val  [n_kernels*k]  kept weights, ascending tap order inside a kernel,
 *                       rounded (nearest even) to compute_dtype;
 *   pid  [n_kernels]    copy of the ids;
 *   ksize 3 only: for each input channel ci a stable counting sort of the
 *   filters by pattern id: perm[ci*Cout+i] = filter at position i,
 *   bucket_off[ci*(P+1)+p] = first position of pattern p (entry P = Cout).
 * n_kernels = Cout*Cin (ksize 3) or floor(Cout*Cin/9) (ksize 1).
 * Precondition: every id in pid_dev is < P (what rtoss_select_patterns writes for the same table).  An id
 * outside the table keeps none of its kernel's weights and its filter is left out of perm (the call stays
 * inside its arrays; the result is then not a valid packed layer).
 * *out must be NULL or an existing handle.  NULL: a new handle is created and
 * its device memory allocated (RTOSS_ERR_ALLOC on failure).  Existing handle
 * of the same layer shape, P, k and dtype: it is re-packed in place without
 * any allocation (the paper re-selects patterns in every pruning iteration);
 * a handle of another shape is RTOSS_ERR_INVALID_ARG.  The work is enqueued
 * on the stream; the handle is usable by later calls on the same stream.
 * Free with rtoss_packed_destroy (which synchronises the device). */
rtoss_status rtoss_pack(rtoss_ctx* ctx, const void* w_dev, rtoss_dtype w_dtype, int Cout, int Cin, int ksize,
                        const uint16_t* masks_host, int P, int k, const uint8_t* pid_dev,
                        rtoss_dtype compute_dtype, rtoss_packed** out, void* cuda_stream);

typedef struct {
    int Cout, Cin, ksize, P, k;
    rtoss_dtype dtype;   /* type of val */
    int64_t n_kernels;   /* entries of pid */
    int64_t n_values;    /* entries of val = n_kernels*k */
} rtoss_packed_info;
rtoss_status rtoss_packed_info_get(const rtoss_packed* p, rtoss_packed_info* info);

/* Copy the canonical arrays to caller-owned host buffers (any may be NULL to
 * skip it).  Sizes: pid n_kernels bytes; val n_values elements of the packed
 * dtype; perm Cin*Cout and bucket_off Cin*(P+1) uint32 (ksize 3 only; ignored
 * for ksize 1).  Synchronises the stream. */
rtoss_status rtoss_packed_export(rtoss_ctx* ctx, const rtoss_packed* p, uint8_t* pid_host, void* val_host,
                                 uint32_t* perm_host, uint32_t* bucket_off_host, void* cuda_stream);

/* Expand to dense masked weights W (.) M ([Cout][Cin][3][3] or [Cout][Cin]) in
 * the packed dtype; pruned positions are +0. */
rtoss_status rtoss_packed_to_dense(rtoss_ctx* ctx, const rtoss_packed* p, void* w_masked_dev, void* cuda_stream);
void rtoss_packed_destroy(rtoss_packed* p);

/* ---- whole-model pruning pass ------------------------------------------------ */

/* The pruning pass visits every convolution layer of the model (the outer loop of Algorithm 1 calling Algorithm 2,
 * or Algorithm 3 for 1x1 layers); a batch runs selection and packing of ALL its layers in two kernel launches.
 * Results are bit-identical to rtoss_select_patterns + rtoss_pack called layer by layer.
 *
 * One item per layer.  `packed` is an existing handle for that layer (made once by rtoss_pack; it owns the
 * device arrays the batch re-writes, so a batch call allocates nothing and may be captured into a CUDA graph).
 * `pid_dev` (nullable, device, Cout*Cin or floor(Cout*Cin/9) bytes) also receives the ids.  `pid_from`: -1, or
 * the index of an EARLIER item of the same shape and table whose patterns this layer inherits (Section IV.A:
 * the layers of a group share the parent's kernel patterns): the selection is then evaluated on that item's
 * weights (on the root of the chain, if that item inherits too) and applied to this layer's own.
 * The arrays w_dev, pid_dev and the handles must stay valid, and the tables unchanged, for the batch's life:
 * rtoss_batch_create copies pointers and tables to the device once (it synchronises); the handles take the
 * batch's tables.  Weights may change between calls -- that is the point: call again after every update.
 * Errors: RTOSS_ERR_INVALID_ARG (null, shape mismatch with the handle, handle used twice, bad pid_from),
 * RTOSS_ERR_BAD_PATTERN_TABLE, RTOSS_ERR_ALIGNMENT (w_dev not 16-byte aligned), RTOSS_ERR_ALLOC. */
typedef struct {
    const void* w_dev; /* [Cout][Cin][3][3] or [Cout][Cin], device */
    rtoss_dtype w_dtype;
    int Cout, Cin, ksize;
    const uint16_t* masks_host; /* P masks of k taps, host */
    int P, k;
    uint8_t* pid_dev;     /* nullable */
    rtoss_packed* packed; /* existing handle of this layer */
    int pid_from;         /* -1 or index of an earlier item */
} rtoss_batch_item;
typedef struct rtoss_batch rtoss_batch;
rtoss_status rtoss_batch_create(rtoss_ctx* ctx, const rtoss_batch_item* items, int L, rtoss_batch** out);
/* Enqueue the pass on the stream: ids, packed values, filter order and the tensor path's weights of every layer. */
rtoss_status rtoss_batch_select_pack(rtoss_ctx* ctx, const rtoss_batch* batch, void* cuda_stream);
/* Frees the batch's own tables (not the handles).  The caller makes sure no call is still running. */
void rtoss_batch_destroy(rtoss_batch* batch);

/* Pruned dense weights with no allocation anywhere (the paper has no counterpart: this entry point
 * exists for deployment, not for the method).  Same result as rtoss_select_patterns followed by
 * rtoss_pack (compute type = w_dtype) and rtoss_packed_to_dense: w_pruned_dev receives W (.) mask,
 * [Cout][Cin][3][3] or [Cout][Cin] in w_dtype, pruned positions +0.  It is meant for callers that
 * cannot call cudaMalloc: a process whose device memory was all handed to its own arena at start-up,
 * or a loop that cannot afford the device-wide synchronisation cudaMalloc / cudaFree imply.  It needs
 * no context and no packed handle and works on the current device.
 *   - The pattern ids, the one intermediate, live in a fixed 1 MiB device array inside the library
 *     (held by every GPU that loads the library until the process exits).  A layer with more than
 *     2^20 kernels (Cout*Cin for ksize 3, floor(Cout*Cin/9) for ksize 1) is refused with
 *     RTOSS_ERR_UNSUPPORTED.
 *   - The first call on a device looks the array's address up (cudaGetSymbolAddress); make that first
 *     call outside any stream capture.
 *   - w_pruned_dev may be w_dev itself (pruning in place, W <- W (.) mask); two different arrays that overlap
 *     are refused with RTOSS_ERR_INVALID_ARG.
 *   - All calls on a device share the array and it keeps the last call's ids.  Each call overwrites
 *     what it reads, so nothing needs clearing, but two calls whose kernels overlap on the GPU (two
 *     streams, two host threads) race on it: keep calls on one device in stream order.
 * Errors: RTOSS_ERR_INVALID_ARG, RTOSS_ERR_BAD_PATTERN_TABLE, RTOSS_ERR_ALIGNMENT (16 bytes),
 * RTOSS_ERR_UNSUPPORTED (too many kernels), RTOSS_ERR_CUDA. */
rtoss_status rtoss_prune_dense_static(const void* w_dev, rtoss_dtype w_dtype, int Cout, int Cin, int ksize,
                                      const uint16_t* masks_host, int P, int k, void* w_pruned_dev, void* cuda_stream);

/* ---- inference convolution over the packed weights ------------------------ */

typedef struct {
    int N, H, W;            /* batch and INPUT height / width */
    int stride;             /* 1 or 2 */
    rtoss_layout layout;    /* of x and y */
    rtoss_dtype io_dtype;   /* of x and y; accumulation is always fp32 */
    rtoss_act act;
    const float* bias_dev;  /* [Cout] fp32, or NULL */
    int y_channel_offset;   /* y may be a channel slice of a wider tensor: */
    int y_channel_stride;   /*   channels of that tensor, 0 = Cout */
    rtoss_path path;        /* which kernel family runs the call */
    const void* residual_dev; /* NULL, or a tensor laid out exactly like y (same type, layout, channel stride and
                               * offset: element (n,co,oy,ox) at the index it has in y) that is added before the
                               * activation: y = act(round(conv + bias) + residual), the sum formed in fp32 and
                               * rounded once more -- for act none and ReLU bit for bit what the convolution with
                               * act = none followed by rtoss_add_act gives, in one pass; for SiLU the same up to
                               * the rounding of the two SiLU evaluations (the residual connection that closes a
                               * bottleneck block; not part of the paper's method).  May be y itself.  Tensor
                               * path only (NHWC; 16-bit data with more than 64 filters or a 3x3 kernel, or fp32 data; pointer 16-byte
                               * aligned): other calls return RTOSS_ERR_UNSUPPORTED before anything is launched
                               * and the caller adds separately. */
    int residual_after_act;   /* 0: as above.  1: the residual is added behind the activation instead,
                               * y = round(act(conv + bias)) + residual, rounded once more: bit for bit (every
                               * activation) what the convolution followed by rtoss_add_act with act = none gives
                               * (the shortcut of a bottleneck block whose last convolution carries the activation). */
} rtoss_conv_desc;

/* y[n,co,oy,ox] = act( bias[co] + sum_ci sum_{t in mask(pid[co,ci])}
 *                      w[co,ci,t] * x[n,ci,oy*s+r-1,ox*s+c-1] ),  t = 3r+c,
 * zero outside the image (padding 1); Ho = (H-1)/s+1, Wo = (W-1)/s+1.  The
 * result is that of the k kept taps per kernel (the cost model of Section II.B
 * counts the non-zero weights).  Both kernel families evaluate it over the
 * dense-expanded weights, pruned taps as zeros: the sparsity saves weight
 * bytes, not multiplications.  x: N x Cin x H x W in the
 * given layout, y: N x Cs x Ho x Wo with Cs = y_channel_stride (or Cout),
 * written at channels [offset, offset+Cout).  x and y must not overlap.  The
 * packed handle must come from rtoss_pack with ksize 3. */
rtoss_status rtoss_conv3x3_pattern(rtoss_ctx* ctx, const rtoss_packed* p, const void* x_dev, void* y_dev,
                                   const rtoss_conv_desc* desc, void* cuda_stream);

/* y[n,co,oy,ox] = act( bias[co] + sum over kept flat positions e = co*Cin+ci
 *                      of w[e] * x[n,ci,oy*s,ox*s] ); position e is kept when
 * it lies in a full run g = e/9 and tap e%9 is in mask(pid[g]) (Section IV.D).
 * No padding; Ho = (H-1)/s+1.  Handle from rtoss_pack with ksize 1. */
rtoss_status rtoss_conv1x1_pattern(rtoss_ctx* ctx, const rtoss_packed* p, const void* x_dev, void* y_dev,
                                   const rtoss_conv_desc* desc, void* cuda_stream);

/* Several INDEPENDENT convolutions at once (no item reads or overwrites what another item writes): the pyramid levels
 * a detection tower is applied to (Section V evaluates RetinaNet, whose towers share their weights across five
 * levels), the two towers, the two 1x1 branches that open a block.  Results are those of the single calls.  Items
 * that qualify for the tensor path with more than 64 filters or a 3x3 kernel, and agree in kernel size, data type
 * and (3x3) stride, share ONE launch, up to twenty at a time: small items then fill the SMs the large ones leave idle
 * instead of paying a launch each.  The other items run as single launches inside the same call.  *launches
 * (nullable) receives the number of kernel launches made.  Errors: those of the single calls; nothing is launched
 * when an argument check fails. */
typedef struct {
    const rtoss_packed* packed; /* ksize 3 or 1 */
    const void* x_dev;
    void* y_dev;
    rtoss_conv_desc desc;
} rtoss_conv_item;
rtoss_status rtoss_conv_group(rtoss_ctx* ctx, const rtoss_conv_item* items, int n, int* launches, void* cuda_stream);

/* Convolutions that DEPEND on one another, in one launch: the three convolutions of a bottleneck block, a whole
 * stage of such blocks, successive layers of the towers (Section V's models are chains of such layers; every launch
 * between two of them costs its start-up and its drain).  items[0..n) are given in an order in which they could run
 * one after the other, n <= 32.  after (n words, or NULL) says which earlier items an item has to wait for: bit j of
 * after[i], j < i, when item i reads what item j writes, or writes where item j reads or writes.  NULL: the library
 * derives exactly that from the address ranges of the items' inputs, outputs and residual operands
 * (rtoss_chain_deps).  The result is that of the single calls issued in the given order.
 *
 * Consecutive items that qualify for a shared launch (tensor path, more than 64 filters or a 3x3 kernel, one data
 * type; at most 20) go out as ONE kernel: its CTAs walk the items' tiles in order and, before the first tile of an
 * item, wait until all tiles of the items it depends on are written (a counter per item in device memory; the wait is
 * bounded like every device-side wait, see rtoss_set_wait_limit, and reports through rtoss_device_status).  Items
 * that do not depend on one another run side by side as in rtoss_conv_group.  Such a launch relies on all its CTAs
 * (at most one per SM) being on the device together: while it runs, no other work may occupy SMs without end, and two
 * such launches must not run concurrently on different streams.  An item that does not qualify, or that has so few
 * tiles and so many input channels that a launch of its own spreads it over more SMs (split along the channels)
 * while the items that could run beside it do not fill the SMs either, runs as a launch of its own between the shared
 * ones (the stream orders them); an item
 * whose desc.path is RTOSS_PATH_TENSOR rather than RTOSS_PATH_AUTO stays in the shared launch whenever it qualifies.  *launches (nullable) receives the number of kernel
 * launches made.
 * Errors: RTOSS_ERR_INVALID_ARG (null items, n outside 1..32, a bit of after[i] at or above i) and those of the single
 * calls; nothing is launched when an argument check fails. */
rtoss_status rtoss_conv_chain(rtoss_ctx* ctx, const rtoss_conv_item* items, int n, const uint32_t* after, int* launches,
                              void* cuda_stream);

/* The dependencies rtoss_conv_chain derives when it is given none (host arithmetic on the pointers; nothing is
 * launched, no device is touched): after[i] gets bit j, j < i, when the input or residual operand of item i overlaps
 * the output buffer of item j, or the output buffer of item i overlaps the input, residual operand or output buffer
 * of item j.  An output buffer counts with its whole pixel pitch (y_channel_stride), so two items that write disjoint
 * channel slices of one buffer are ordered too.  n <= 32. */
rtoss_status rtoss_chain_deps(const rtoss_conv_item* items, int n, uint32_t* after);
/* The same rule on plain byte ranges: spans holds, per item, {x_lo, x_hi, y_lo, y_hi, r_lo, r_hi} (half-open ranges;
 * an absent residual operand is an empty range).  RTOSS_ERR_INVALID_ARG for a null pointer, n outside 1..32 or a
 * range whose end lies before its start. */
rtoss_status rtoss_chain_deps_spans(const uint64_t* spans, int n, uint32_t* after);

/* The tensor path (RTOSS_PATH_TENSOR, or RTOSS_PATH_AUTO when it applies) takes: NHWC, stride 1 or 2, io_dtype equal
 * to the packed dtype; bf16 / fp16 with Cin a multiple of 8, or fp32 with Cin a multiple of 4.  fp32 data is computed
 * with tf32 instructions on values split into a 19-bit head and a remainder (three products per tap, fp32
 * accumulation): results stay within the fp32 bound of 1e-4 of max(|y|, rms(y)) and cost six times the tensor time of
 * 16-bit data.  It multiplies blocks of 128 filters x 16
 * channels per tap on the tensor cores and leaves out the blocks in which every weight is pruned (none with
 * per-kernel patterns on ordinary weights; 9 - k of every 9 with rtoss_select_patterns_shared); inside a block the
 * pruned taps are multiplied as zeros.  Results agree with the FMA path to fp32 summation order.
 *
 * Device-side waits of that path are bounded.  If one runs out, the kernel records a non-zero code in
 * the context and returns; rtoss_device_status synchronises the device, reports the code
 * (RTOSS_ERR_TIMEOUT when non-zero) and clears it. */
rtoss_status rtoss_device_status(rtoss_ctx* ctx, int* code);

/* Limit of those waits in SM clock cycles (default 2e9, about a second; at least 1000). */
rtoss_status rtoss_set_wait_limit(rtoss_ctx* ctx, long long sm_cycles);

/* Failure-detection aid: the NEXT tensor-path launch of this context withholds its first weight copy, so that the
 * waits that depend on it run out and the timeout path above can be exercised.  Nothing illegal happens on the
 * device: every role of the kernel gives up after the wait limit and the kernel ends normally; the output of that
 * call is undefined.  Only a launch of a single CTA (one tile) is accepted -- any other returns RTOSS_ERR_CUDA
 * without launching -- and the request is consumed either way.  Lower the wait limit first. */
rtoss_status rtoss_inject_lost_copy(rtoss_ctx* ctx);

/* Same convolutions with HOST buffers: copies x to the device, runs the
 * kernel for the handle's ksize, copies y back and waits for it.  x_host and
 * y_host are dense tensors in desc's layout and dtype (y_channel_* apply).  The batch is cut into chunks of
 * images whose copies and kernels overlap on three internal streams; pinned host memory is needed for
 * the copies to be asynchronous.
 * Uses (and grows on demand) the context's device workspace, so concurrent
 * calls on one context are not allowed.  bias_dev stays a device pointer.
 * The kernels run on the context's own (non-blocking) streams, which are not ordered after the stream
 * rtoss_pack was given: the handle's packing must have COMPLETED (synchronise that stream, or an event)
 * before this call. */
rtoss_status rtoss_conv_pattern_host(rtoss_ctx* ctx, const rtoss_packed* p, const void* x_host, void* y_host,
                                     const rtoss_conv_desc* desc);

/* How the FMA path would tile a 3x3 call (host arithmetic only, nothing is launched; for Cin <= 4 only small_cin is
 * set: that kernel has no staging plan).  staging: 0 = plain loads, 1 = NCHW rows as aligned vectors of vector_bytes
 * through cp.async, 2 = NHWC pixels as 16-byte vectors through cp.async.  With staging 1 the address of every vector,
 *   ((n*Cin + ci)*H*W + iy*W + tx*lanes_x*pixels_per_lane*stride - vector_bytes/es + j*vector_bytes/es) * es
 * (es = bytes per activation, tx = tile column, j = vector inside the staged row), is a multiple of vector_bytes for a
 * 16-byte aligned tensor: the plan guarantees it, and the CPU tests check it tile by tile.  Not part of the paper's
 * method.  RTOSS_ERR_INVALID_ARG, RTOSS_ERR_UNSUPPORTED (no shape fits the shared memory). */
typedef struct {
    int small_cin;
    int pixels_per_lane, filters_per_warp, warps, ctas_per_sm; /* kernel shape */
    int lanes_x, lanes_y;                                      /* lane arrangement inside a warp */
    int tiles_x, tiles_y, grid_x, grid_y;                      /* tiles per image, CTAs */
    int staged_rows, staged_cols;                              /* input tile with halo */
    int staging, vector_bytes, vectors_per_plane;
    int shared_bytes;
} rtoss_fma_plan;
rtoss_status rtoss_fma_plan3x3(const rtoss_conv_desc* desc, int Cin, int Cout, int k, rtoss_dtype packed_dtype,
                               rtoss_fma_plan* out);

/* The tensor path's tiling of a call, host arithmetic only (nothing is launched, no device is touched): what the
 * launcher of a single call would choose for a layer of this shape on a device of sm_count SMs (0: 148).  desc gives N,
 * H, W, stride, layout and whether there is a residual operand (any non-null residual_dev; it is not dereferenced).
 * eligible = 0 when the tensor path does not take the shape (then the rest is zero).  Lets the CPU tests check the
 * planner's invariants -- shared memory within an SM's, at most 256 positions and 256 box elements per dimension,
 * stage sizes multiples of the swizzle atom -- and shows how a layer is cut.  Not part of the paper's method.
 * RTOSS_ERR_INVALID_ARG for a null pointer or a size below 1. */
typedef struct {
    int eligible;
    int rows_per_tile, cols_per_tile, pitch, positions;      /* output rows and columns of a tile, position pitch, the MMA's N */
    int staged_rows, sub_tiles;                              /* input rows staged per tile; 4 parity sub-tiles for 3x3 stride 2 */
    int act_stages, weight_stages, taps_per_weight_stage;    /* ring depths; taps fetched by one bulk copy */
    int row_bytes, act_stage_bytes, weight_stage_bytes;      /* 128, or 64 for 16-bit layers of at most 32 input channels */
    int shared_bytes;
    int positions_on_m;                                      /* narrow 1x1 layers */
    int split_k;                                             /* CTAs of a cluster sharing a tile's channel blocks (1: none) */
    int tiles;
} rtoss_tensor_plan;
rtoss_status rtoss_tensor_plan_of(const rtoss_conv_desc* desc, int ksize, int Cin, int Cout, rtoss_dtype dtype, int sm_count,
                                  rtoss_tensor_plan* out);

/* ---- glue between the convolutions of a whole network ---------------------- */
/* Not part of the paper's method (Table 3 and Fig. 6 time whole models, whose graphs need these between the
 * pruned convolutions).  Element-wise, bandwidth-bound; x and y in the given layout and dtype; y may be a
 * channel slice [offset, offset + C) of a tensor with y_channel_stride channels (0 = C), which makes a
 * concatenation a write.  Errors: RTOSS_ERR_INVALID_ARG, RTOSS_ERR_CUDA. */

/* k x k max-pooling, given stride and padding (pad <= k/2; padded positions never win):
 * Ho = (H + 2*pad - k)/stride + 1. */
rtoss_status rtoss_maxpool2d(const void* x_dev, void* y_dev, int N, int C, int H, int W, int k, int stride, int pad,
                             rtoss_layout layout, rtoss_dtype dtype, int y_channel_offset, int y_channel_stride,
                             void* cuda_stream);
/* Nearest-neighbour up-sampling by 2: y[n,c,oh,ow] = x[n,c,oh/2,ow/2], output 2H x 2W. */
rtoss_status rtoss_upsample2x(const void* x_dev, void* y_dev, int N, int C, int H, int W, rtoss_layout layout,
                              rtoss_dtype dtype, int y_channel_offset, int y_channel_stride, void* cuda_stream);
/* y = act(a + b) over n_elements contiguous elements (residual connections); the sum is formed in fp32 and
 * rounded once.  y may alias a or b. */
rtoss_status rtoss_add_act(const void* a_dev, const void* b_dev, void* y_dev, int64_t n_elements, rtoss_dtype dtype,
                           rtoss_act act, void* cuda_stream);

#ifdef __cplusplus
}
#endif
#endif /* RTOSS_H */
