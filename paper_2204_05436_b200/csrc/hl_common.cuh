// Shared declarations of the Hotline sm_100a library: context layout, status word, remap probe.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>
#include <stddef.h>

#include "hotline.h"

namespace hl {

constexpr int kSMsFallback = 148;          // used only if the device's SM count cannot be queried (B200: 2 x 74)
constexpr int kRemapRowsPerBlock = 224;    // 7 bitmap words per 32-byte remap block
constexpr int kSortTile = 2048;            // keys per radix-sort tile (256 threads x 8)
constexpr int kScanTile = 2048;            // elements per scan tile (256 threads x 8)
constexpr int kSelTile = 4096;             // rows per hot-set selection tile (256 threads x 16)
constexpr int kBwdChunk = 32;              // sorted lookups per backward chunk
constexpr int kMoverCtasDefault = 16;      // working CTAs of a host-link mover inside a schedule: write-backs
constexpr int kReadCtasDefault = 24;       // ... and host reads (a wider read finishes sooner and costs the step nothing)
// Per-mini-batch kernels are launched with one CTA per tile of work rather than as chip-filling persistent grids:
// they run next to the host-link movers of another micro-batch, which slow down the SMs they sit on, and the
// hardware block scheduler then simply hands those SMs fewer CTAs.
constexpr int kMaxGrid = 1 << 22;

// One 32-byte sector per 224 rows: w[0] = number of popular rows before this block, w[1..7] = hit bitmap.
struct __align__(32) RemapBlock {
    uint32_t w[8];
};

// State of the count-threshold selection (device memory).
struct SelectState {
    unsigned long long hist[256];
    unsigned long long k_remaining;    // rows still wanted among the current prefix class
    unsigned long long quota_eq;       // rows with count == threshold to keep (in ascending id)
    unsigned long long total;          // lookups counted so far
    unsigned int prefix;               // high digits of the threshold found so far
    unsigned int mask;                 // bits of `prefix` that are fixed
    unsigned int c_min;                // smallest admissible count (>= 1)
    unsigned int threshold;            // final: k-th largest admissible count
    int take_all;                      // fewer admissible rows than wanted: keep them all
};

struct Regions {
    // common
    int32_t* status;                   // [8]  status[0] = first device error
    int64_t* table_base;               // [T+1]
    unsigned char** table_ptrs;        // [T] host-memory base of every table (hl_set_host_tables), device copy
    RemapBlock* remap;                 // [n_remap_blocks]
    // profile
    uint32_t* counts;                  // [N]
    SelectState* sel;
    uint32_t* sel_gt;                  // [n_sel_tiles + 1]
    uint32_t* sel_eq;                  // [n_sel_tiles + 1]
    // fragment
    uint8_t* frag_flags;               // [max_batch]
    int32_t* frag_scan;                // [max_bags + 1]
    int32_t* frag_tiles;               // [scan tiles + 1]
    // backward
    int32_t* bwd_keys[2];              // [max_nnz]
    int32_t* bwd_vals[2];              // [max_nnz]
    uint32_t* bwd_hist;                // [256 * sort tiles]
    float* bwd_part;                   // [2 * n_chunks * D]
    int32_t* bwd_n;                    // [4] lookups in the micro-batch
    // cold
    int32_t* cold_keys[2];
    int32_t* cold_vals[2];
    uint32_t* cold_hist;
    int32_t* cold_rank;                // [max_nnz + 1]
    int32_t* cold_tiles;               // [scan tiles + 1]
    int32_t* cold_n;                   // [4] cold lookups
};

}  // namespace hl

struct hl_ctx {
    int32_t T, D, S;
    int64_t N;
    int32_t max_batch;
    int64_t max_nnz, max_bags;
    int64_t hot_cap, staging_cap;
    int64_t n_remap_blocks, n_sel_tiles;
    int device;
    int sms;                           // multiprocessors of `device` (queried at hl_create)
    int mover_ctas, scatter_ctas;      // working CTAs of the host-link movers inside a schedule (hl_set_mover_ctas)
    int fwd_ctas, bwd_ctas;            // CTAs per multiprocessor of the forward / backward-sum kernel (0 = default)
    int cold_cluster;                  // CTAs of the one-cluster cold-row search (0 = not asked yet; 8 or 16)
    int test_poll_limit;               // > 0: poll limit of the bounded device waits (hl_test_bounded_waits)
    int64_t test_stall_tile;           // with it: the tile / mover stage that never delivers (-1: none)
    int64_t* h_table_base;             // host copy [T+1]
    int per_table;                     // 1: the host table is one allocation per table (r.table_ptrs is set)
    hl::Regions r;
    int timing_on;                     // optional kernel timers (hl_timing_enable)
    cudaEvent_t timer[HL_TIMER_COUNT][2];
    // optional observer of the kernel timers' marks (the pipeline's trace): called with (user, which, end, stream)
    void (*mark_hook)(void*, int, int, cudaStream_t);
    void* mark_user;
};

// Context of the wide-id index path (hl_wide_*): global row ids are 64-bit, every table still has fewer than 2^31
// rows.  Popularity is counted in a hashed counter and the popular rows are found through a hashed remap, so nothing
// here is sized by the number of rows.
struct hl_wide {
    int32_t T, S;
    int64_t N;
    int32_t max_batch;
    int64_t max_nnz, max_bags, hot_cap, staging_cap;
    int64_t counter_slots, remap_slots;     // powers of two
    int sms;
    int64_t* h_table_base;
    // device regions (carved from the caller's workspace)
    int32_t* status;
    int64_t* table_base;                     // [T+1]
    long long* c_keys;                       // [counter_slots] row id or -1
    uint32_t* c_cnt;                         // [counter_slots]
    hl::SelectState* sel;
    uint32_t *sel_gt, *sel_eq;               // [counter_slots / kSelTile + 2]
    int32_t* n_seen;                         // [4]
    int32_t *e_tab, *e_idx;                  // [counter_slots] table and table-local index of every counted row
    uint32_t *e_cnt, *s_cnt;                 // [counter_slots] its count; the counts in row order
    int32_t* s_ent;                          // [counter_slots] entry behind every position of the row order
    int32_t* sel_idx;                        // [hot_cap] selected positions
    long long* r_keys;                       // [remap_slots] popular row or -1
    int32_t* r_vals;                         // [remap_slots] its slot
    int32_t* sort_keys[2];                   // [max(counter_slots, max_nnz)]
    int32_t* sort_vals[2];
    uint32_t* sort_hist;
    uint8_t* frag_flags;                     // [max_batch]
    int32_t *frag_scan, *frag_tiles;
    int32_t *cold_tab, *cold_idx, *cold_pos; // [max_nnz] cold lookups: table, index, position in X
    int32_t *cold_rank, *cold_tiles, *cold_n;
};

namespace hl {

#define HL_CUDA_TRY(expr)                         \
    do {                                          \
        cudaError_t e__ = (expr);                 \
        if (e__ != cudaSuccess) return HL_ECUDA;  \
    } while (0)

#define HL_LAUNCH_CHECK()                                  \
    do {                                                   \
        if (cudaGetLastError() != cudaSuccess) return HL_ECUDA; \
    } while (0)

// Records the start/end event of one of the optional kernel timers on `stream` (no-op unless enabled).
inline void timer_mark(hl_ctx* ctx, int which, int end, cudaStream_t stream) {
    if (ctx->timing_on && ctx->timer[which][end]) cudaEventRecord(ctx->timer[which][end], stream);
    if (ctx->mark_hook) ctx->mark_hook(ctx->mark_user, which, end, stream);
}

inline int ctx_sms(const hl_ctx* ctx) { return ctx->sms > 0 ? ctx->sms : kSMsFallback; }
// CTAs per multiprocessor of the two bandwidth-bound kernels (hl_set_kernel_width; defaults chosen by measurement)
// (rows of up to 128 fp32: the forward kernel is held to 64 registers, so four of its CTAs fit a multiprocessor)
inline int fwd_ctas_per_sm(const hl_ctx* ctx) { return ctx->fwd_ctas > 0 ? ctx->fwd_ctas : (ctx->D <= 128 ? 4 : 3); }
inline int bwd_ctas_per_sm(const hl_ctx* ctx) { return ctx->bwd_ctas > 0 ? ctx->bwd_ctas : 6; }

__device__ __forceinline__ void set_status(int32_t* status, int32_t code) {
    atomicCAS(status, 0, code);
}

// Hit test only: one 4-byte load.
__device__ __forceinline__ bool remap_hit(const RemapBlock* __restrict__ remap, int64_t g) {
    const uint32_t blk = (uint32_t)(g / kRemapRowsPerBlock);
    const uint32_t r = (uint32_t)(g - (int64_t)blk * kRemapRowsPerBlock);
    const uint32_t word = __ldg(&remap[blk].w[1 + (r >> 5)]);
    return (word >> (r & 31)) & 1u;
}

// Slot of global row g, or -1: one 32-byte sector.
__device__ __forceinline__ int32_t remap_slot(const RemapBlock* __restrict__ remap, int64_t g) {
    const uint32_t blk = (uint32_t)(g / kRemapRowsPerBlock);
    const uint32_t r = (uint32_t)(g - (int64_t)blk * kRemapRowsPerBlock);
    const uint4 lo = __ldg(reinterpret_cast<const uint4*>(&remap[blk].w[0]));
    const uint4 hi = __ldg(reinterpret_cast<const uint4*>(&remap[blk].w[4]));
    const uint32_t w[8] = {lo.x, lo.y, lo.z, lo.w, hi.x, hi.y, hi.z, hi.w};
    const uint32_t wi = 1 + (r >> 5), bit = r & 31;
    uint32_t slot = w[0];
    uint32_t word = 0;
#pragma unroll
    for (uint32_t i = 1; i < 8; ++i) {
        if (i < wi) slot += __popc(w[i]);
        if (i == wi) word = w[i];
    }
    if (!((word >> bit) & 1u)) return -1;
    slot += __popc(word & ((1u << bit) - 1u));
    return (int32_t)slot;
}

// Where the host-DRAM table's rows are: one allocation holding all tables back to back (ptrs == nullptr: row g at
// single + g * row_bytes), or one allocation per table (the address registers of the paper's Data Dispatcher,
// Section V-A): row g of table t at ptrs[t] + (g - base[t]) * row_bytes.
struct TableMap {
    unsigned char* single;
    unsigned char* const* ptrs;
    const int64_t* base;               // [T+1]
    int T;
};

__device__ __forceinline__ unsigned char* row_address(const TableMap& m, int64_t g, int row_bytes) {
    if (m.ptrs == nullptr) return m.single + g * row_bytes;
    int lo = 0, hi = m.T;              // base[lo] <= g < base[hi]
    while (hi - lo > 1) {
        const int mid = (lo + hi) >> 1;
        if (__ldg(&m.base[mid]) <= g) lo = mid;
        else hi = mid;
    }
    return m.ptrs[lo] + (g - __ldg(&m.base[lo])) * row_bytes;
}

// ---- the hashed lookup structures of the wide-id path (global row ids beyond 2^31, hl_wide_*) ------------------
// Randomizer of Section V-C on a 64-bit row id: a 4-round Feistel network on its 32-bit halves (a bijection, so
// distinct rows never collide before the reduction to the table size), round function (x * 0x9E3779B1 + K_r)
// rotated by 15 bits.
__host__ __device__ __forceinline__ uint64_t randomize64(uint64_t g) {
    uint32_t l = (uint32_t)(g >> 32), r = (uint32_t)g;
    const uint32_t k[4] = {0x85EBCA6Bu, 0xC2B2AE35u, 0x27D4EB2Fu, 0x165667B1u};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        uint32_t f = r * 0x9E3779B1u + k[i];
        f = (f << 15) | (f >> 17);
        const uint32_t nl = r;
        r = l ^ f;
        l = nl;
    }
    return ((uint64_t)l << 32) | r;
}

// Open-addressing table row id -> value (linear probing from randomize64(row) & mask; an empty entry holds -1).
struct HashProbe {
    const long long* keys;
    const int32_t* vals;
    uint64_t mask;
    __device__ __forceinline__ int32_t slot(int64_t g) const {
        uint64_t h = randomize64((uint64_t)g) & mask;
        for (uint64_t tries = 0; tries <= mask; ++tries) {
            const long long k = __ldg(&keys[h]);
            if (k == g) return __ldg(&vals[h]);
            if (k < 0) return -1;
            h = (h + 1) & mask;
        }
        return -1;
    }
    __device__ __forceinline__ bool hit(int64_t g) const { return slot(g) >= 0; }
};

// The dense form used by the 32-bit path: one 32-byte block per 224 rows (see RemapBlock).
struct BitmapProbe {
    const RemapBlock* remap;
    __device__ __forceinline__ int32_t slot(int64_t g) const { return remap_slot(remap, g); }
    __device__ __forceinline__ bool hit(int64_t g) const { return remap_hit(remap, g); }
};

__device__ __forceinline__ unsigned lanemask_lt() {
    unsigned m;
    asm("mov.u32 %0, %%lanemask_lt;" : "=r"(m));
    return m;
}

// How long the bounded device-side waits poll before they give up (HL_ETIMEOUT), and -- for the tests of that
// path only -- which tile of a chained scan or sort pass publishes nothing, so that the tiles behind it wait in vain
// (-1: none).  Production value: about a second of polling, far beyond any wait that can occur.
struct WaitCfg {
    int max_polls = 1 << 20;
    int64_t stall_tile = -1;
};
inline WaitCfg wait_cfg(const hl_ctx* ctx) {
    WaitCfg w;
    if (ctx->test_poll_limit > 0) {
        w.max_polls = ctx->test_poll_limit;
        w.stall_tile = ctx->test_stall_tile;
    }
    return w;
}

// ---- primitives implemented in hl_prims.cu -----------------------------------------------------------------
// Exclusive scan of in[0 .. n) into out[0 .. n] (out[n] = total); n = *d_n if d_n != nullptr (clamped to
// n_max), else n_max.  in may alias out.  tiles: scratch of scan_tile_words(n_max) ints.  A chain poll that
// gives up records HL_ETIMEOUT in *status.
int32_t exclusive_scan_i32(const int32_t* in, int32_t* out, const int32_t* d_n, int64_t n_max, int32_t* tiles,
                           int32_t* status, cudaStream_t stream, WaitCfg w = WaitCfg());

// Stable LSD radix sort of (key, value) pairs by the low key_bits bits of the non-negative keys.
// n = *d_n (clamped to n_max).  Returns in *out_keys / *out_vals which of the two buffers holds the result.
int32_t radix_sort_pairs(int32_t* keys[2], int32_t* vals[2], const int32_t* d_n, int64_t n_max, int key_bits,
                         uint32_t* hist, int32_t* status, int32_t** out_keys, int32_t** out_vals,
                         cudaStream_t stream, WaitCfg w = WaitCfg());

// The same from the device (one thread calls; the launches run after the calling grid, in order: see hl_prims.cu).
// radix_sort_pairs_tail returns which buffer (0 / 1) will hold the result.
__device__ int radix_sort_pairs_tail(int32_t* keys0, int32_t* keys1, int32_t* vals0, int32_t* vals1, int64_t n,
                                     int key_bits, uint32_t* hist, int32_t* status, int max_polls);
__device__ void exclusive_scan_i32_tail(const int32_t* in, int32_t* out, int64_t n, int32_t* tiles, int32_t* status,
                                        int max_polls);

// 32-bit words of histogram scratch radix_sort_pairs needs for at most max_nnz pairs.
constexpr int64_t sort_hist_words(int64_t max_nnz) {
    const int64_t n_tiles = ((max_nnz > 0 ? max_nnz : 1) + kSortTile - 1) / kSortTile;
    return 4 * 256 + 8 + 4 * n_tiles * 256;   // digit counts, tickets, tile status words for up to 4 passes
}

// ints behind the backward's partial sums: count words + (chunk, key, last chunk of the run or -1, unused) per chunk
// of kBwdChunk sorted lookups.
constexpr int64_t bwd_span_list_words(int64_t max_nnz) {
    return 8 + 4 * (((max_nnz > 0 ? max_nnz : 1) + kBwdChunk - 1) / kBwdChunk);
}

// where those ints start
inline int32_t* span_count_of(const hl_ctx* ctx) {
    const int64_t max_chunks = ((ctx->max_nnz > 0 ? ctx->max_nnz : 1) + kBwdChunk - 1) / kBwdChunk;
    return reinterpret_cast<int32_t*>(ctx->r.bwd_part + 2 * max_chunks * ctx->D);
}

// ints of scratch exclusive_scan_i32 needs for at most n_max elements (64-bit ticket + status words).
constexpr int64_t scan_tile_words(int64_t n_max) { return 2 * ((n_max > 0 ? n_max : 1) / kScanTile + 3); }

// Selection of the rows with the k largest counts (implemented in hl_profile.cu; see there).
int32_t select_rows_by_count(const uint32_t* counts, int64_t n, SelectState* sel, uint32_t* sel_gt, uint32_t* sel_eq,
                             long long k, long long share_num, long long share_den, int64_t cap, int32_t* out_idx,
                             int64_t* d_n_out, int32_t* status, int sms, cudaStream_t stream);

// Process-wide count of kernels this library has launched (read by hl_launch_count).
void note_launches(int n);

inline int64_t div_up(int64_t a, int64_t b) { return (a + b - 1) / b; }
inline int grid_for(int64_t work_items, int per_block, int max_blocks) {
    int64_t b = div_up(work_items, per_block);
    if (b < 1) b = 1;
    if (b > max_blocks) b = max_blocks;
    return (int)b;
}

}  // namespace hl
