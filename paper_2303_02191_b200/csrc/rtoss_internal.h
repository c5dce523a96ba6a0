// Internal definitions shared by the translation units of librtoss.
#ifndef RTOSS_INTERNAL_H
#define RTOSS_INTERNAL_H

#include <cstddef>
#include <cstdint>

#include "rtoss.h"

// Host-side cache of encoded TMA descriptors (encoding costs microseconds per call).
struct rtoss_tmap_entry {
    const void* base;
    int dims[6];  // what the descriptor was encoded for
    int valid;
    alignas(64) unsigned char map[128];
};

constexpr int kHostChunks = 8;  // the host-buffer path cuts a batch into at most this many chunks

// Launches that carry dependent convolutions count completed problems in device memory: a block of
// RTOSS_CHAIN_SLOT_WORDS words per launch (one per problem and one exit counter, zero between launches), taken in
// turn from RTOSS_CHAIN_SLOTS blocks of the context.
constexpr int RTOSS_CHAIN_SLOTS = 64;
constexpr int RTOSS_CHAIN_SLOT_WORDS = 32;

struct rtoss_ctx {
    int device;
    int sm_count;
    char err[256];
    // device workspace of the host-buffer path (grown on demand)
    void* ws_x;
    size_t ws_x_bytes;
    void* ws_y;
    size_t ws_y_bytes;
    void* h_stream;  // cudaStream_t owned by the context: copies in of the host-buffer path
    void* h_stream2;  // its kernels
    void* h_stream3;  // its copies out
    void* h_ev_in[8];   // cudaEvent_t per batch chunk: copy in done
    void* h_ev_run[8];  // kernel done
    int* dev_status;  // device word: 0, or the code of a bounded device-side wait that ran out
    long long wait_cycles;     // limit of every device-side wait of the tensor path, in SM clock cycles
    mutable int inject_next;   // failure-detection test hook: the next tensor-path launch withholds its first weight copy
    mutable rtoss_tmap_entry tmap_cache[32];  // activation descriptors of the tensor path, round robin
    mutable int tmap_next;
    unsigned* chain_done;      // device: RTOSS_CHAIN_SLOTS x RTOSS_CHAIN_SLOT_WORDS completion counters, all zero at rest
    mutable int chain_next;    // the block the next launch with dependent convolutions takes
};

struct rtoss_packed {
    int device;
    int Cout, Cin, ksize, P, k;
    rtoss_dtype dtype;
    int64_t n_kernels;
    uint8_t* pid;          // [n_kernels]
    void* val;             // [n_kernels*k] in dtype
    uint32_t* perm;        // [Cin*Cout]      (ksize 3)
    uint32_t* bucket_off;  // [Cin*(P+1)]     (ksize 3)
    uint16_t* masks_dev;   // [256]
    void* wtc;             // tensor path: dense-expanded weights [taps][Cout][Cin] in dtype, or NULL
    unsigned long long* issue;  // tensor path, ksize 3: per (tile of 128 filters, block of 64 channels) which (tap, 16-channel
                                // slab) pairs hold any kept weight (bit 4*tap + slab); [issue_n] words, or NULL
    int issue_n;
    mutable rtoss_tmap_entry wtc_map;  // its TMA descriptor, encoded at first use
    uint16_t masks[256];
};

// Pattern table passed by value to kernels (constant bank, uniform reads).
struct MaskTable {
    uint16_t m[256];
};

bool rtoss_table_ok(const uint16_t* masks, int P, int k);

// Makes `device` current for the life of the object and gives the caller its own current device back afterwards:
// an entry point must not leave another GPU selected behind the back of the caller (or of torch).  Defined in
// rtoss_api.cu (host code, CUDA runtime).
struct rtoss_device_guard {
    explicit rtoss_device_guard(int device);
    ~rtoss_device_guard();
    rtoss_device_guard(const rtoss_device_guard&) = delete;
    rtoss_device_guard& operator=(const rtoss_device_guard&) = delete;
    int prev;
    bool switched;
};

static inline size_t rtoss_dtype_size(rtoss_dtype d) { return d == RTOSS_F32 ? 4 : 2; }

// Layout of the tensor path's dense-expanded weights wtc[tap][row][ci].  Normally row = filter (rows = Cout).  A
// narrow 3x3 layer (Cout <= 64) stores its filters `copies` times down 128 rows, copy c of filter co at row
// c*rep_rows + co (rows in between stay zero): the MMA then fills all 128 accumulator lanes with outputs and every
// epilogue warp has lanes to read.
struct rtoss_wtc_layout {
    int rows, rep_rows, copies;
};
static inline rtoss_wtc_layout rtoss_wtc_layout_of(int Cout, int ksize) {
    rtoss_wtc_layout l;
    if (ksize == 3 && Cout <= 64) {
        l.rep_rows = Cout <= 32 ? 32 : 64;
        l.rows = 128;
        l.copies = 128 / l.rep_rows;
    } else {
        l.rows = Cout;
        l.rep_rows = Cout;
        l.copies = 1;
    }
    return l;
}

// kernel launchers (select_pack.cu, conv3x3_alu.cu, conv1x1_alu.cu); each returns a cudaError_t as int
int rtoss_launch_select(const void* w, rtoss_dtype wdt, int64_t n_kernels, const MaskTable& t, int P, uint8_t* pid,
                        void* stream);
int rtoss_launch_pack_values(const void* w, rtoss_dtype wdt, int64_t n_kernels, const MaskTable& t, const uint8_t* pid,
                             int k, void* val, rtoss_dtype vdt, uint8_t* pid_copy, void* wtc, int ksize, int Cout, int Cin,
                             void* stream);
int rtoss_launch_pack_order(const uint8_t* pid, int Cout, int Cin, int P, uint32_t* perm, uint32_t* bucket_off,
                            const uint16_t* masks_dev, unsigned long long* issue, int cb_log2, void* stream);
int rtoss_launch_select_shared(const void* w, rtoss_dtype wdt, int Cout, int Cin, int FB, int CB, const MaskTable& t, int P,
                               uint8_t* pid, void* stream);
int rtoss_launch_to_dense(const rtoss_packed* p, void* w_out, void* stream);
int rtoss_launch_pid_histogram(const uint8_t* pid, int64_t n, int P, unsigned long long* counts, void* stream);
int rtoss_launch_conv3x3(const rtoss_ctx* ctx, const rtoss_packed* p, const void* x, void* y,
                         const rtoss_conv_desc* d, void* stream);
int rtoss_launch_conv1x1(const rtoss_ctx* ctx, const rtoss_packed* p, const void* x, void* y,
                         const rtoss_conv_desc* d, void* stream);
// Number of issue words of a layer (tiles of 128 filter rows x blocks of 64 channels).
static inline int rtoss_issue_cb_log2(rtoss_dtype d) { return d == RTOSS_F32 ? 5 : 6; }   // channels per 128-byte block
static inline int rtoss_issue_words(int Cout, int Cin, int ksize, rtoss_dtype d) {
    const int cb = 1 << rtoss_issue_cb_log2(d);
    return ((rtoss_wtc_layout_of(Cout, ksize).rows + 127) / 128) * ((Cin + cb - 1) / cb);
}

// tensor path (conv_tc.cu)
bool rtoss_tc_weights_eligible(const rtoss_packed* p);
bool rtoss_tc_eligible(const rtoss_packed* p, const rtoss_conv_desc* d, const void* x, const void* y);
int rtoss_launch_conv_tc(const rtoss_ctx* ctx, const rtoss_packed* p, const void* x, void* y,
                         const rtoss_conv_desc* d, void* stream);
bool rtoss_tc_groupable(const rtoss_packed* p, const rtoss_conv_desc* d, const void* x, const void* y);
// several independent convolutions in one launch: 0 = launched, -1 = the set cannot share a launch (nothing launched)
int rtoss_launch_conv_tc_group(const rtoss_ctx* ctx, int n, const rtoss_packed* const* ps, const void* const* xs,
                               void* const* ys, const rtoss_conv_desc* const* ds, void* stream);
// the same with dependencies: bit j of after[i] = convolution i waits (inside the launch) for convolution j < i
int rtoss_launch_conv_tc_chain(const rtoss_ctx* ctx, int n, const rtoss_packed* const* ps, const void* const* xs,
                               void* const* ys, const rtoss_conv_desc* const* ds, const uint32_t* after, void* stream);
int rtoss_tc_max_problems();   // most convolutions one launch carries
// a launch of its own would cut this call along K (few tiles, many channel blocks); a shared launch never does
bool rtoss_tc_prefers_split(const rtoss_ctx* ctx, const rtoss_packed* p, const rtoss_conv_desc* d, long* tiles_out);

#endif
