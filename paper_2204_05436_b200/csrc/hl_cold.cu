// The non-popular micro-batch's working set: classify its lookups, find the distinct cold rows, stage them from
// the host-DRAM table (bulk copies over the host link, row by row) behind the hot cache, and write them back.
#include "hl_common.cuh"
#include <cooperative_groups.h>

namespace hl {
namespace {

constexpr int kThreads = 256;

// Lookups of X: popular rows resolve to their cache slot at once; cold ones are appended (row, position) to
// the list that is sorted next.  Append order is arbitrary; the sort and the final slots do not depend on it.
__global__ void __launch_bounds__(kThreads) k_cold_classify(int32_t* __restrict__ ids,
                                                            const int32_t* __restrict__ offsets,
                                                            const int32_t* __restrict__ d_n_non, int max_batch,
                                                            int bags_per_sample_all, int64_t cap_ids, int64_t N,
                                                            const RemapBlock* __restrict__ remap,
                                                            int32_t* __restrict__ keys, int32_t* __restrict__ vals,
                                                            int32_t* __restrict__ d_n_cold_lookups, int64_t max_nnz,
                                                            int32_t* status) {
    int n_non = *d_n_non;
    n_non = n_non < 0 ? 0 : (n_non > max_batch ? max_batch : n_non);
    int64_t L = offsets[(int64_t)n_non * bags_per_sample_all];
    if (L > cap_ids) L = cap_ids;
    const unsigned lt = lanemask_lt();
    const int64_t stride = (int64_t)gridDim.x * blockDim.x;
    // whole warps iterate together (the ballot below needs every lane)
    for (int64_t j0 = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) & ~int64_t(31); j0 < L; j0 += stride) {
        const int64_t j = j0 + (threadIdx.x & 31);
        bool cold = false;
        int32_t g = -1;
        if (j < L) {
            g = ids[j];
            if (g >= N) {
                set_status(status, HL_EBOUNDS);
                ids[j] = -1;
            } else if (g >= 0) {
                const int32_t slot = remap_slot(remap, g);
                if (slot >= 0) ids[j] = slot;
                else cold = true;
            }
        }
        const unsigned vote = __ballot_sync(0xffffffffu, cold);
        if (vote) {
            int32_t base = 0;
            if ((threadIdx.x & 31) == 0) base = atomicAdd(d_n_cold_lookups, __popc(vote));
            base = __shfl_sync(0xffffffffu, base, 0);
            if (cold) {
                const int64_t pos = (int64_t)base + __popc(vote & lt);
                if (pos < max_nnz) {
                    keys[pos] = g;
                    vals[pos] = (int32_t)j;
                }
            }
        }
    }
}

__global__ void __launch_bounds__(kThreads) k_cold_heads(const int32_t* __restrict__ keys, int64_t n,
                                                         int32_t* __restrict__ heads) {
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (int64_t)gridDim.x * blockDim.x)
        heads[i] = (i == 0 || keys[i] != keys[i - 1]) ? 1 : 0;
}

// rank_excl[i] = number of run heads before i; the row at i has rank rank_excl[i] if it is a head, else
// rank_excl[i] - 1.  A row of rank r is staged at cache slot slot0 + r (slot0 = start of the staging window).
__global__ void __launch_bounds__(kThreads) k_cold_assign(const int32_t* __restrict__ keys,
                                                          const int32_t* __restrict__ vals, int64_t n,
                                                          const int32_t* __restrict__ rank_excl, int64_t slot0,
                                                          int64_t staging_cap, int32_t* __restrict__ ids,
                                                          int32_t* __restrict__ cold_rows,
                                                          int64_t* __restrict__ d_n_cold, int32_t* status,
                                                          int64_t cap_ids) {
    if (blockIdx.x == 0 && threadIdx.x == 0) {
        int64_t distinct = rank_excl[n];
        if (distinct > staging_cap) {
            set_status(status, HL_ECAPACITY);
            distinct = staging_cap;
        }
        *d_n_cold = distinct;
    }
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (int64_t)gridDim.x * blockDim.x) {
        const bool head = i == 0 || keys[i] != keys[i - 1];
        const int64_t rank = head ? rank_excl[i] : rank_excl[i] - 1;
        const int64_t where = vals[i];
        if (where < 0 || where >= cap_ids || rank < 0) continue;   // only after a chain poll gave up (HL_ETIMEOUT)
        if (rank < staging_cap) {
            if (head) cold_rows[rank] = keys[i];
            ids[where] = (int32_t)(slot0 + rank);
        } else {
            ids[where] = -1;   // no room to stage this row: the lookup is dropped and the status word says so
        }
    }
}

// ---- few cold lookups: one thread-block cluster does sort, distinct-row ranking and slot assignment ----------------
// With at most CTAS * kSmallPerCta cold lookups (a DLRM-large mini-batch has about 18 K) the chain of radix passes,
// head flags, scan and assignment -- nine launches that each take longer to start than to run -- is one kernel of
// one cluster of CTAS CTAs: 16 (40 960 lookups; a cluster size the kernel has to opt in to) where the device can
// place such a cluster, else 8 (20 480).  CTA c owns positions [c * kSmallPerCta, (c + 1) * kSmallPerCta) of the list.  Every pass ranks
// the pairs, held in registers, by one digit (per-warp digit counters, as in the tile kernel of the general sort),
// adds up the digit counts of the cluster's CTAs through distributed shared memory, and writes each pair into the shared
// memory of the CTA that owns its new position.  The sorted list is then ranked and assigned in place.
// Order of a CTA's items: position = warp * (32 * kSmallItems) + round * 32 + lane.
// Larger inputs: the kernel launches the general path itself (tile sort, head flags, scan, assignment) as tail
// launches, which run after this grid and before anything the host queued behind it -- so the host queues the same
// two kernels for every mini-batch and never needs to know which path ran.  *d_n_general = the number of cold lookups
// handed to the general path (0: none).
constexpr int kSmallThreads = 256;
constexpr int kSmallItems = 10;
constexpr int kSmallPerCta = kSmallThreads * kSmallItems;       // 2560
constexpr int kSmallWarps = kSmallThreads / 32;

// what the general path works on (device pointers into the context's cold region)
struct GeneralArgs {
    int32_t* keys[2];
    int32_t* vals[2];
    uint32_t* hist;
    int32_t* rank;
    int32_t* tiles;
    int64_t cap_ids;
    int key_bits;
    int max_polls;
};

__device__ __forceinline__ int block_scan_small(int v, int* smem33, int& total) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    int incl = v;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
        const int o = __shfl_up_sync(0xffffffffu, incl, d);
        if (lane >= d) incl += o;
    }
    if (lane == 31) smem33[warp] = incl;
    __syncthreads();
    if (warp == 0) {
        const int w = lane < kSmallWarps ? smem33[lane] : 0;
        int wi = w;
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
            const int o = __shfl_up_sync(0xffffffffu, wi, d);
            if (lane >= d) wi += o;
        }
        if (lane < kSmallWarps) smem33[lane] = wi - w;
        if (lane == 31) smem33[32] = wi;
    }
    __syncthreads();
    const int res = smem33[warp] + incl - v;
    total = smem33[32];
    __syncthreads();
    return res;
}

template <int CTAS>
__global__ void __launch_bounds__(kSmallThreads) k_cold_small(const int32_t* __restrict__ keys_in,
                                                              const int32_t* __restrict__ vals_in,
                                                              const int32_t* __restrict__ d_n, int64_t n_max,
                                                              int passes, int64_t slot0, int64_t staging_cap,
                                                              int32_t* __restrict__ ids,
                                                              int32_t* __restrict__ cold_rows,
                                                              int64_t* __restrict__ d_n_cold,
                                                              int32_t* __restrict__ d_n_general, int32_t* status,
                                                              GeneralArgs ga) {
    namespace cg = cooperative_groups;
    cg::cluster_group cluster = cg::this_cluster();
    __shared__ int32_t s_key[kSmallPerCta];
    __shared__ int32_t s_val[kSmallPerCta];
    __shared__ uint32_t cnt[kSmallWarps * 256];
    __shared__ uint32_t cta_hist[256];       // this CTA's digit counts, read by the other CTAs
    __shared__ uint32_t digit_base[256];
    __shared__ int cta_heads;                // this CTA's number of run heads, read by the other CTAs
    __shared__ int scan_smem[33];
    int64_t n64 = d_n[0];
    n64 = n64 < 0 ? 0 : (n64 < n_max ? n64 : n_max);
    const int cta = (int)cluster.block_rank();
    if (n64 > CTAS * kSmallPerCta) {         // the same decision in all CTAs, before any cluster barrier
        if (cta == 0 && threadIdx.x == 0) {
            d_n_general[0] = (int32_t)n64;
            // the general path, queued behind this grid: stable sort of the (row, position) pairs by row, a flag at
            // the head of every run, ranks by a scan of the flags, slots and distinct rows from the ranks
            const int cur = radix_sort_pairs_tail(ga.keys[0], ga.keys[1], ga.vals[0], ga.vals[1], n64, ga.key_bits,
                                                  ga.hist, status, ga.max_polls);
            const int32_t* sk = ga.keys[cur];
            const int32_t* sv = ga.vals[cur];
            int64_t grid = (n64 + kThreads - 1) / kThreads;
            grid = grid < 2048 ? grid : 2048;
            k_cold_heads<<<(unsigned)grid, kThreads, 0, cudaStreamTailLaunch>>>(sk, n64, ga.rank);
            exclusive_scan_i32_tail(ga.rank, ga.rank, n64, ga.tiles, status, ga.max_polls);
            k_cold_assign<<<(unsigned)grid, kThreads, 0, cudaStreamTailLaunch>>>(
                sk, sv, n64, ga.rank, slot0, staging_cap, ids, cold_rows, d_n_cold, status, ga.cap_ids);
            if (cudaGetLastError() != cudaSuccess) set_status(status, HL_ECUDA);
        }
        return;
    }
    if (cta == 0 && threadIdx.x == 0) d_n_general[0] = 0;
    const int n = (int)n64;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const unsigned lt = lanemask_lt();
    const int cta_base = cta * kSmallPerCta;
    const int warp_base = warp * (32 * kSmallItems);
    int32_t key[kSmallItems];
    uint32_t aux[kSmallItems];        // low 16 bits: where the pair's value sits in vals_in; high 16: rank in its warp
#pragma unroll
    for (int r = 0; r < kSmallItems; ++r) {
        const int idx = cta_base + warp_base + r * 32 + lane;
        key[r] = idx < n ? keys_in[idx] : 0x7fffffff;     // padding sorts behind every row id and stays there
        aux[r] = (uint32_t)idx;
    }
    for (int p = 0; p < passes; ++p) {
        const int shift = 8 * p;
        for (int i = threadIdx.x; i < kSmallWarps * 256; i += kSmallThreads) cnt[i] = 0;
        __syncthreads();
#pragma unroll
        for (int r = 0; r < kSmallItems; ++r) {
            const uint32_t d = ((uint32_t)key[r] >> shift) & 255u;
            const unsigned peers = __match_any_sync(0xffffffffu, d);
            const uint32_t before = cnt[warp * 256 + d];
            __syncwarp();
            aux[r] = (aux[r] & 0xffffu) | ((before + __popc(peers & lt)) << 16);
            if ((peers & lt) == 0) cnt[warp * 256 + d] = before + __popc(peers);
            __syncwarp();
        }
        __syncthreads();
        {   // thread d: prefix of digit d over this CTA's warps; publish the CTA's count
            const int d = threadIdx.x;
            uint32_t total = 0;
#pragma unroll
            for (int w = 0; w < kSmallWarps; ++w) {
                const uint32_t c = cnt[w * 256 + d];
                cnt[w * 256 + d] = total;
                total += c;
            }
            cta_hist[d] = total;
        }
        cluster.sync();     // all counts published; all CTAs have taken the previous pass's pairs out of shared memory
        {
            const int d = threadIdx.x;
            uint32_t before_me = 0, all_ctas = 0;
#pragma unroll
            for (int c = 0; c < CTAS; ++c) {
                const uint32_t v = *cluster.map_shared_rank(&cta_hist[d], c);
                if (c < cta) before_me += v;
                all_ctas += v;
            }
            int whole;
            const int smaller = block_scan_small((int)all_ctas, scan_smem, whole);     // pairs with a smaller digit
            digit_base[d] = (uint32_t)smaller + before_me;
        }
        __syncthreads();
#pragma unroll
        for (int r = 0; r < kSmallItems; ++r) {
            const uint32_t d = ((uint32_t)key[r] >> shift) & 255u;
            const uint32_t pos = digit_base[d] + cnt[warp * 256 + d] + (aux[r] >> 16);
            const unsigned owner = pos / kSmallPerCta, off = pos % kSmallPerCta;
            *cluster.map_shared_rank(&s_key[off], owner) = key[r];
            *cluster.map_shared_rank(&s_val[off], owner) = (int32_t)(aux[r] & 0xffffu);
        }
        cluster.sync();     // every pair has arrived
#pragma unroll
        for (int r = 0; r < kSmallItems; ++r) {
            const int idx = warp_base + r * 32 + lane;
            key[r] = s_key[idx];
            aux[r] = (uint32_t)s_val[idx];
        }
    }
    // The sorted pairs are in the CTAs' shared memory (the last barrier above made them visible).  Thread t of CTA c
    // ranks positions cta_base + [t * kSmallItems, (t + 1) * kSmallItems).
    const int i0 = threadIdx.x * kSmallItems;
    int32_t mine[kSmallItems + 1];           // mine[0] = the key before my first position
    mine[0] = -1;
    if (i0 > 0) mine[0] = s_key[i0 - 1];
    else if (cta > 0) mine[0] = *cluster.map_shared_rank(&s_key[kSmallPerCta - 1], cta - 1);
    int32_t where[kSmallItems];
    int heads = 0;
#pragma unroll
    for (int u = 0; u < kSmallItems; ++u) {
        const int i = cta_base + i0 + u;
        mine[u + 1] = s_key[i0 + u];
        where[u] = i < n ? vals_in[s_val[i0 + u]] : -1;          // the lookup's position in X's ids
        if (i < n && (i == 0 || mine[u + 1] != mine[u])) ++heads;
    }
    int cta_total;
    int rank = block_scan_small(heads, scan_smem, cta_total);    // heads before my first position, within the CTA
    if (threadIdx.x == 0) cta_heads = cta_total;
    cluster.sync();
    int distinct = 0;
#pragma unroll
    for (int c = 0; c < CTAS; ++c) {
        const int v = *cluster.map_shared_rank(&cta_heads, c);
        if (c < cta) rank += v;
        distinct += v;
    }
    if (cta == 0 && threadIdx.x == 0) {
        int64_t dn = distinct;
        if (dn > staging_cap) {
            set_status(status, HL_ECAPACITY);
            dn = staging_cap;
        }
        *d_n_cold = dn;
    }
#pragma unroll
    for (int u = 0; u < kSmallItems; ++u) {
        const int i = cta_base + i0 + u;
        if (i < n) {
            const bool head = i == 0 || mine[u + 1] != mine[u];
            const int my_rank = head ? rank : rank - 1;
            if (head) ++rank;
            if (my_rank < staging_cap) {
                if (head) cold_rows[my_rank] = mine[u + 1];
                ids[where[u]] = (int32_t)(slot0 + my_rank);
            } else {
                ids[where[u]] = -1;     // no room to stage this row: the lookup is dropped, the status word says so
            }
        }
    }
    cluster.sync();     // no CTA leaves while another may still read its shared memory
}

// dst[(dst_row0 + i), :] = table[rows[i], :] (or the other way round); G lanes per row, UR rows in flight per
// group.  Rows i with skip[i] >= 0 are left alone.
template <int G, bool TO_TABLE>
__global__ void __launch_bounds__(kThreads) k_move_rows(float* __restrict__ dense_side, int64_t dense_row0,
                                                        TableMap table, const int32_t* __restrict__ rows,
                                                        const int64_t* __restrict__ d_n, int64_t n_max,
                                                        int64_t table_rows, int D4,
                                                        const int32_t* __restrict__ skip, int32_t* status) {
    constexpr int UR = 16;
    int64_t n = *d_n;
    n = n < 0 ? 0 : (n < n_max ? n : n_max);
    const int sub = threadIdx.x % G;
    const int64_t group = ((int64_t)blockIdx.x * kThreads + threadIdx.x) / G;
    const int64_t n_groups = (int64_t)gridDim.x * kThreads / G;
    float4* dense4 = reinterpret_cast<float4*>(dense_side) + dense_row0 * D4;
    for (int64_t i0 = group * UR; i0 < n; i0 += n_groups * UR) {
        float4* trow[UR];              // the row in the host table, nullptr = nothing to move
#pragma unroll
        for (int u = 0; u < UR; ++u) {
            int64_t g = i0 + u < n ? (int64_t)rows[i0 + u] : -1;
            if (skip != nullptr && g >= 0 && skip[i0 + u] >= 0) g = -1;   // row comes from elsewhere
            if (g >= table_rows) {
                set_status(status, HL_EBOUNDS);
                g = -1;
            }
            trow[u] = g >= 0 ? reinterpret_cast<float4*>(row_address(table, g, D4 * 16)) : nullptr;
        }
        for (int c = sub; c < D4; c += G) {
            float4 v[UR];
#pragma unroll
            for (int u = 0; u < UR; ++u)
                if (trow[u]) v[u] = TO_TABLE ? dense4[(i0 + u) * D4 + c] : trow[u][c];
#pragma unroll
            for (int u = 0; u < UR; ++u)
                if (trow[u]) {
                    if (TO_TABLE) trow[u][c] = v[u];
                    else dense4[(i0 + u) * D4 + c] = v[u];
                }
        }
    }
}

// src[i] = position of rows[i] in the ascending list prev[0 .. *d_n_prev), or -1.
__global__ void __launch_bounds__(kThreads) k_cold_match(const int32_t* __restrict__ rows,
                                                         const int64_t* __restrict__ d_n, int64_t n_max,
                                                         const int32_t* __restrict__ prev,
                                                         const int64_t* __restrict__ d_n_prev, int64_t n_prev_max,
                                                         int32_t* __restrict__ src) {
    int64_t n = *d_n, np = *d_n_prev;
    n = n < 0 ? 0 : (n < n_max ? n : n_max);
    np = np < 0 ? 0 : (np < n_prev_max ? np : n_prev_max);
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (int64_t)gridDim.x * blockDim.x) {
        const int32_t g = rows[i];
        int64_t lo = 0, hi = np;
        while (lo < hi) {
            const int64_t mid = (lo + hi) >> 1;
            if (prev[mid] < g) lo = mid + 1;
            else hi = mid;
        }
        src[i] = (lo < np && prev[lo] == g) ? (int32_t)lo : -1;
    }
}

// cache[to_row0 + i, :] = cache[from_row0 + src[i], :] for every i < *d_n with src[i] >= 0.
template <int G>
__global__ void __launch_bounds__(kThreads) k_forward_rows(float* cache, int64_t from_row0, int64_t to_row0,
                                                           const int32_t* __restrict__ src,
                                                           const int64_t* __restrict__ d_n, int64_t n_max, int D4) {
    int64_t n = *d_n;
    n = n < 0 ? 0 : (n < n_max ? n : n_max);
    const int sub = threadIdx.x % G;
    const int64_t group = ((int64_t)blockIdx.x * kThreads + threadIdx.x) / G;
    const int64_t n_groups = (int64_t)gridDim.x * kThreads / G;
    float4* c4 = reinterpret_cast<float4*>(cache);
    for (int64_t i = group; i < n; i += n_groups) {
        const int32_t j = src[i];
        if (j < 0 || j >= n_max) continue;
        for (int c = sub; c < D4; c += G) c4[(to_row0 + i) * D4 + c] = c4[(from_row0 + j) * D4 + c];
    }
}

// ---- row mover on the bulk-copy (TMA) engine ----------------------------------------------------------------
// The same copy as k_move_rows, issued as asynchronous bulk copies: every row is one cp.async.bulk from its
// source into shared memory (completion counted in bytes on an mbarrier) and one cp.async.bulk from shared memory
// to its destination.  The rows in flight are then requests of the copy engine of the SM, not pending loads of
// its load-store unit, so that embedding-bag CTAs of another micro-batch that share the SM keep their own
// loads moving while hundreds of host rows, each waiting microseconds for its address translation, are pending.
// Source, destination and row size are multiples of 16 bytes (dim % 4 == 0, 16-byte aligned bases).
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void bulk_load(void* smem_dst, const void* gmem_src, uint32_t bytes, uint64_t* mbar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
                     smem_u32(smem_dst)),
                 "l"(gmem_src), "r"(bytes), "r"(smem_u32(mbar))
                 : "memory");
}
__device__ __forceinline__ void bulk_store(void* gmem_dst, const void* smem_src, uint32_t bytes) {
    asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;" ::"l"(gmem_dst),
                 "r"(smem_u32(smem_src)), "r"(bytes)
                 : "memory");
}

constexpr int kBulkThreads = 128;
constexpr int kBulkStages = 2;
constexpr int kBulkStageBytes = 16384;
constexpr int kBulkMaxPolls = 1 << 22;
constexpr int kBulkStagesPerCta = 16;     // stages of rows per working CTA before another CTA joins in
// Working CTAs of the mover inside a schedule (hl_set_mover_ctas changes it per context).  16 CTAs x 2 stages x
// 16 KB keep 512 KB of rows in flight: 16 K rows of 256 bytes take about 150 us to read and 120 us to write back
// next to the other streams' kernels.  More CTAs move the rows faster (about 100 us with 2 per SM, alone), fewer
// slower (one CTA writes back 64 rows every 3.4 us); what a transfer costs the kernels that run next to it hardly
// depends on that, so the host read, which nothing else of its mini-batch waits for at once, runs on 24 CTAs (about
// 135 us) and the write-back on 16.  (The hot-cache load of hl_build_remap and hl_flush_hot, which run alone, use
// 2 CTAs per SM and reach 90 % of the memcpy rate.)  The defaults, kReadCtasDefault and kMoverCtasDefault, are set at
// hl_create.

// What a launch of the mover needs to know about its context.
struct MoveCfg {
    int sms;            // multiprocessors of the device: the launch has at most 2 CTAs per SM
    int min_ctas;       // CTAs that work however few rows there are
    int max_polls;      // poll limit of the wait for a stage to fill
    int stall;          // tests only: CTA 0 issues no loads for its first stage, whose wait then runs out
};

template <bool TO_TABLE>
__global__ void __launch_bounds__(kBulkThreads) k_move_rows_bulk(float* dense_side, int64_t dense_row0, TableMap table,
                                                                 const int32_t* __restrict__ rows,
                                                                 const int64_t* __restrict__ d_n, int64_t n_max,
                                                                 int64_t table_rows, int row_bytes,
                                                                 int rows_per_stage,
                                                                 const int32_t* __restrict__ skip, int32_t* status,
                                                                 int min_ctas, int max_polls, int stall) {
    __shared__ __align__(128) unsigned char stage[kBulkStages][kBulkStageBytes];
    __shared__ __align__(8) uint64_t mbar[kBulkStages];
    __shared__ unsigned int stage_bytes[kBulkStages];
    __shared__ int s_gave_up;
    int64_t n = *d_n;
    n = n < 0 ? 0 : (n < n_max ? n : n_max);
    const int tid = threadIdx.x;
    if (tid == 0) {
        for (int s = 0; s < kBulkStages; ++s) {
            asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(&mbar[s])), "r"(1) : "memory");
            stage_bytes[s] = 0;
        }
        s_gave_up = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    unsigned char* dense = reinterpret_cast<unsigned char*>(dense_side) + dense_row0 * row_bytes;
    const int64_t n_batches = (n + rows_per_stage - 1) / rows_per_stage;
    // The launch has as many CTAs as the largest transfer could use; how many of them work is decided here, from the
    // number of rows there really are: min_ctas for a mini-batch's worth of a DLRM-sized model (more would only slow
    // the kernels that run beside the mover), up to all of them when a mini-batch moves hundreds of thousands of rows
    // (the link is then all that matters): one more CTA for every kBulkStagesPerCta stages of rows.
    int64_t active = n_batches / kBulkStagesPerCta;
    active = active < min_ctas ? min_ctas : active;
    active = active < (int64_t)gridDim.x ? active : (int64_t)gridDim.x;
    if ((int64_t)blockIdx.x >= active) return;
    int it = 0;
    for (int64_t b = blockIdx.x; b < n_batches; b += active, ++it) {
        const int s = it % kBulkStages;
        const uint32_t parity = (uint32_t)(it / kBulkStages) & 1u;
        const int64_t i0 = b * rows_per_stage;
        const int cnt = (int)min((int64_t)rows_per_stage, n - i0);
        // this thread's earlier stores out of stage s have finished reading shared memory
        asm volatile("cp.async.bulk.wait_group.read %0;" ::"n"(kBulkStages - 1) : "memory");
        __syncthreads();
        // which of my rows move, and how many bytes the stage expects
        unsigned int my_bytes = 0;
        for (int r = tid; r < cnt; r += kBulkThreads) {
            const int64_t g = rows[i0 + r];
            const bool ok = g >= 0 && g < table_rows && !(skip != nullptr && skip[i0 + r] >= 0);
            if (g >= table_rows) set_status(status, HL_EBOUNDS);
            if (ok) my_bytes += (unsigned int)row_bytes;
        }
        if (my_bytes) atomicAdd(&stage_bytes[s], my_bytes);
        __syncthreads();
        if (tid == 0) {
            asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(&mbar[s])),
                         "r"(stage_bytes[s])
                         : "memory");
            stage_bytes[s] = 0;
        }
        const bool stalled = stall && blockIdx.x == 0 && it == 0;     // tests: the expected bytes never arrive
        for (int r = tid; r < cnt && !stalled; r += kBulkThreads) {
            const int64_t g = rows[i0 + r];
            const bool ok = g >= 0 && g < table_rows && !(skip != nullptr && skip[i0 + r] >= 0);
            if (!ok) continue;
            const unsigned char* src = TO_TABLE ? dense + (i0 + r) * row_bytes : row_address(table, g, row_bytes);
            bulk_load(&stage[s][r * row_bytes], src, (uint32_t)row_bytes, &mbar[s]);
        }
        // wait for the stage to fill (bounded)
        uint32_t done = 0;
        for (int polls = 0; !done; ++polls) {
            asm volatile(
                "{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
                : "=r"(done)
                : "r"(smem_u32(&mbar[s])), "r"(parity)
                : "memory");
            if (!done && polls > max_polls) {
                set_status(status, HL_ETIMEOUT);
                s_gave_up = 1;
                break;
            }
        }
        // A wait that ran out ends this CTA's work: the stage is not written, no further stage is started (its
        // barrier phases would be out of step), and the CTA leaves once its earlier stores have completed.  The rows
        // it was responsible for stay unmoved; the status word says so.
        __syncthreads();
        if (s_gave_up) break;
        for (int r = tid; r < cnt; r += kBulkThreads) {
            const int64_t g = rows[i0 + r];
            const bool ok = g >= 0 && g < table_rows && !(skip != nullptr && skip[i0 + r] >= 0);
            if (!ok) continue;
            unsigned char* dst = TO_TABLE ? row_address(table, g, row_bytes) : dense + (i0 + r) * row_bytes;
            bulk_store(dst, &stage[s][r * row_bytes], (uint32_t)row_bytes);
        }
        asm volatile("cp.async.bulk.commit_group;" ::: "memory");
    }
    asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
    if (s_gave_up) {
        // loads of the abandoned stage that are still on their way get a bounded grace period to land before the
        // shared memory goes back to the SM
        for (int i = 0; i < 64; ++i) __nanosleep(1000);
    }
}

template <bool TO_TABLE>
int32_t launch_move_rows(float* dense_side, int64_t dense_row0, TableMap table, const int32_t* rows,
                         const int64_t* d_n, int64_t n_max, int64_t table_rows, int D, const int32_t* skip,
                         MoveCfg cfg, int32_t* status, cudaStream_t stream) {
    if (n_max <= 0) return HL_OK;
    const int D4 = D / 4;
    const int row_bytes = D * 4;
    if (row_bytes <= kBulkStageBytes) {
        const int rows_per_stage = kBulkStageBytes / row_bytes;
        const int grid = grid_for(n_max, rows_per_stage, 2 * cfg.sms);
        k_move_rows_bulk<TO_TABLE><<<grid, kBulkThreads, 0, stream>>>(
            dense_side, dense_row0, table, rows, d_n, n_max, table_rows, row_bytes, rows_per_stage, skip, status,
            cfg.min_ctas < grid ? cfg.min_ctas : grid, cfg.max_polls, cfg.stall);
        note_launches(1);
        HL_LAUNCH_CHECK();
        return HL_OK;
    }
    // Rows wider than a stage of the bulk mover (16 KB): plain 128-bit loads and stores, 48 CTAs x 16 groups x 16 rows
    // in flight on a third of the SMs, so that the kernels of the other streams keep CTA slots.
    const int grid = 48;
    if (D4 <= 4)
        k_move_rows<4, TO_TABLE><<<grid, kThreads, 0, stream>>>(dense_side, dense_row0, table, rows, d_n, n_max,
                                                               table_rows, D4, skip, status);
    else if (D4 <= 8)
        k_move_rows<8, TO_TABLE><<<grid, kThreads, 0, stream>>>(dense_side, dense_row0, table, rows, d_n, n_max,
                                                               table_rows, D4, skip, status);
    else if (D4 <= 16)
        k_move_rows<16, TO_TABLE><<<grid, kThreads, 0, stream>>>(dense_side, dense_row0, table, rows, d_n, n_max,
                                                                table_rows, D4, skip, status);
    else
        k_move_rows<32, TO_TABLE><<<grid, kThreads, 0, stream>>>(dense_side, dense_row0, table, rows, d_n, n_max,
                                                                table_rows, D4, skip, status);
    note_launches(1);
    HL_LAUNCH_CHECK();
    return HL_OK;
}

int bits_for(int64_t max_value) {
    int b = 1;
    while ((int64_t(1) << b) <= max_value) ++b;
    return b;
}

}  // namespace

// the host table as the movers see it: `host_table` itself, or the per-table allocations installed by
// hl_set_host_tables (then `host_table` only says that there is a table)
static TableMap table_map(const hl_ctx* ctx, const float* host_table) {
    TableMap m;
    m.single = reinterpret_cast<unsigned char*>(const_cast<float*>(host_table));
    m.ptrs = ctx->per_table ? ctx->r.table_ptrs : nullptr;
    m.base = ctx->r.table_base;
    m.T = ctx->T;
    return m;
}

// how the movers of this context are launched: inside a schedule (`width` = the context's setting) or alone on the
// chip (`width` = 0: two CTAs per SM, the link's full rate)
static MoveCfg move_cfg(const hl_ctx* ctx, int width) {
    MoveCfg c;
    c.sms = ctx_sms(ctx);
    c.min_ctas = width > 0 ? width : 2 * c.sms;
    c.max_polls = ctx->test_poll_limit > 0 ? ctx->test_poll_limit : kBulkMaxPolls;
    c.stall = ctx->test_poll_limit > 0 && ctx->test_stall_tile >= 0;
    return c;
}

int32_t launch_gather_rows(hl_ctx* ctx, float* dst, int64_t dst_row0, const float* table, const int32_t* rows,
                           const int64_t* d_n, int64_t n_max, int32_t* status, cudaStream_t stream) {
    // loading the hot cache happens with nothing else on the chip: two mover CTAs per SM, for the link's full rate
    return launch_move_rows<false>(dst, dst_row0, table_map(ctx, table), rows, d_n, n_max, ctx->N, ctx->D, nullptr,
                                   move_cfg(ctx, 0), status, stream);
}

}  // namespace hl

using namespace hl;

namespace hl {
namespace {

// Shared body of hl_gather_cold and hl_gather_cold_ahead.  Staging window: cache slots
// [hot_cap + stage_row0, hot_cap + stage_row0 + stage_rows).
// First half of the cold-row search: classify X's lookups, then the one-cluster kernel, which either finishes the
// search or launches the general path behind itself; cold_n[1] says which (0, or the number of cold lookups).
int32_t index_begin(hl_ctx* ctx, hl_ubatch* non, const int32_t* d_n_non, int64_t stage_row0, int64_t stage_rows,
                    int32_t* d_cold_rows, int64_t* d_n_cold, cudaStream_t stream) {
    Regions& r = ctx->r;
    if (ctx->max_nnz == 0) {
        HL_CUDA_TRY(cudaMemsetAsync(d_n_cold, 0, sizeof(int64_t), stream));
        HL_CUDA_TRY(cudaMemsetAsync(r.cold_n, 0, 4 * sizeof(int32_t), stream));
        return HL_OK;
    }
    if (!non->ids) return HL_EINVAL;
    HL_CUDA_TRY(cudaMemsetAsync(r.cold_n, 0, 4 * sizeof(int32_t), stream));
    const int grid = grid_for(ctx->max_nnz, kThreads, 4 * ctx_sms(ctx));
    k_cold_classify<<<grid, kThreads, 0, stream>>>(non->ids, non->offsets, d_n_non, ctx->max_batch, ctx->T * ctx->S,
                                                   non->cap_ids, ctx->N, r.remap, r.cold_keys[0], r.cold_vals[0],
                                                   r.cold_n, ctx->max_nnz, r.status);
    note_launches(1);
    HL_LAUNCH_CHECK();
    const int key_bits = bits_for(ctx->N - 1);
    GeneralArgs ga;
    for (int i = 0; i < 2; ++i) {
        ga.keys[i] = r.cold_keys[i];
        ga.vals[i] = r.cold_vals[i];
    }
    ga.hist = r.cold_hist;
    ga.rank = r.cold_rank;
    ga.tiles = r.cold_tiles;
    ga.cap_ids = non->cap_ids;
    ga.key_bits = key_bits;
    ga.max_polls = wait_cfg(ctx).max_polls;
    // the widest cluster the device can place: 16 CTAs (a non-portable size) or 8; asked once per context
    if (ctx->cold_cluster == 0) {
        ctx->cold_cluster = 8;
        cudaLaunchConfig_t probe = {};
        probe.gridDim = dim3(16);
        probe.blockDim = dim3(kSmallThreads);
        cudaLaunchAttribute pa[1];
        pa[0].id = cudaLaunchAttributeClusterDimension;
        pa[0].val.clusterDim.x = 16;
        pa[0].val.clusterDim.y = pa[0].val.clusterDim.z = 1;
        probe.attrs = pa;
        probe.numAttrs = 1;
        int clusters = 0;
        if (cudaFuncSetAttribute(k_cold_small<16>, cudaFuncAttributeNonPortableClusterSizeAllowed, 1) == cudaSuccess &&
            cudaOccupancyMaxActiveClusters(&clusters, k_cold_small<16>, &probe) == cudaSuccess && clusters >= 1)
            ctx->cold_cluster = 16;
        (void)cudaGetLastError();
    }
    const int ctas = ctx->cold_cluster;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(ctas);
    cfg.blockDim = dim3(kSmallThreads);
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = ctas;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    HL_CUDA_TRY(cudaLaunchKernelEx(&cfg, ctas == 16 ? k_cold_small<16> : k_cold_small<8>,
                                   (const int32_t*)r.cold_keys[0], (const int32_t*)r.cold_vals[0],
                                   (const int32_t*)r.cold_n, ctx->max_nnz, (key_bits + 7) / 8,
                                   ctx->hot_cap + stage_row0, stage_rows, non->ids, d_cold_rows, d_n_cold,
                                   r.cold_n + 1, r.status, ga));
    note_launches(1);
    HL_LAUNCH_CHECK();
    return HL_OK;
}

// Second half: the match against the previous mini-batch's cold rows.  (Whatever the search needed beyond its
// one-cluster kernel was launched by that kernel and has run by the time anything queued here starts.)
int32_t index_end(hl_ctx* ctx, int64_t stage_rows, int32_t* d_cold_rows, int64_t* d_n_cold,
                  const int32_t* d_prev_rows, const int64_t* d_n_prev, int32_t* d_fwd_src, cudaStream_t stream) {
    if (ctx->max_nnz == 0) return HL_OK;
    if (d_prev_rows) {
        k_cold_match<<<grid_for(stage_rows, kThreads, 2 * ctx_sms(ctx)), kThreads, 0, stream>>>(
            d_cold_rows, d_n_cold, stage_rows, d_prev_rows, d_n_prev, ctx->staging_cap, d_fwd_src);
        note_launches(1);
        HL_LAUNCH_CHECK();
    }
    return HL_OK;
}

int32_t gather_impl(hl_ctx* ctx, hl_ubatch* non, const int32_t* d_n_non, const float* host_table, float* d_cache,
                    int64_t stage_row0, int64_t stage_rows, int32_t* d_cold_rows, int64_t* d_n_cold,
                    const int32_t* d_prev_rows, const int64_t* d_n_prev, int32_t* d_fwd_src,
                    cudaEvent_t record_after_index, cudaEvent_t wait_a, cudaEvent_t wait_b, bool do_index,
                    bool do_move, cudaStream_t stream) {
    Regions& r = ctx->r;
    if (!do_index) {
        if (ctx->max_nnz == 0) return HL_OK;
        timer_mark(ctx, HL_TIMER_GATHER_MOVE, 0, stream);
        const int32_t st = launch_move_rows<false>(d_cache, ctx->hot_cap + stage_row0,
                                                   table_map(ctx, host_table), d_cold_rows, d_n_cold, stage_rows,
                                                   ctx->N, ctx->D, d_fwd_src, move_cfg(ctx, ctx->mover_ctas), r.status,
                                                   stream);
        timer_mark(ctx, HL_TIMER_GATHER_MOVE, 1, stream);
        return st;
    }
    int32_t st = index_begin(ctx, non, d_n_non, stage_row0, stage_rows, d_cold_rows, d_n_cold, stream);
    if (st != HL_OK) return st;
    st = index_end(ctx, stage_rows, d_cold_rows, d_n_cold, d_prev_rows, d_n_prev, d_fwd_src, stream);
    if (st != HL_OK) return st;
    if (record_after_index) HL_CUDA_TRY(cudaEventRecord(record_after_index, stream));
    if (!do_move) return HL_OK;
    if (wait_a) HL_CUDA_TRY(cudaStreamWaitEvent(stream, wait_a, 0));
    if (wait_b) HL_CUDA_TRY(cudaStreamWaitEvent(stream, wait_b, 0));
    timer_mark(ctx, HL_TIMER_GATHER_MOVE, 0, stream);
    st = launch_move_rows<false>(d_cache, ctx->hot_cap + stage_row0, table_map(ctx, host_table), d_cold_rows,
                                 d_n_cold, stage_rows, ctx->N, ctx->D, d_prev_rows ? d_fwd_src : nullptr,
                                 move_cfg(ctx, ctx->mover_ctas), r.status, stream);
    timer_mark(ctx, HL_TIMER_GATHER_MOVE, 1, stream);
    return st;
}

bool window_ok(const hl_ctx* ctx, int64_t row0, int64_t rows) {
    return row0 >= 0 && rows >= 0 && row0 + rows <= ctx->staging_cap;
}

}  // namespace
}  // namespace hl

extern "C" int32_t hl_gather_cold(hl_ctx* ctx, hl_ubatch* non, const int32_t* d_n_non, const float* host_table,
                                  float* d_cache, int32_t* d_cold_rows, int64_t* d_n_cold, void* stream_) {
    if (!ctx || !non || !non->offsets || !d_n_non || !host_table || !d_cache || !d_cold_rows || !d_n_cold)
        return HL_EINVAL;
    return gather_impl(ctx, non, d_n_non, host_table, d_cache, 0, ctx->staging_cap, d_cold_rows, d_n_cold, nullptr,
                       nullptr, nullptr, nullptr, nullptr, nullptr, true, true, static_cast<cudaStream_t>(stream_));
}

extern "C" int32_t hl_gather_cold_ahead(hl_ctx* ctx, hl_ubatch* non, const int32_t* d_n_non, const float* host_table,
                                        float* d_cache, int64_t stage_row0, int64_t stage_rows, int32_t* d_cold_rows,
                                        int64_t* d_n_cold, const int32_t* d_prev_cold_rows, const int64_t* d_n_prev,
                                        int32_t* d_fwd_src, void* record_after_index, void* wait_before_move_a,
                                        void* wait_before_move_b, void* stream_) {
    if (!ctx || !non || !non->offsets || !d_n_non || !host_table || !d_cache || !d_cold_rows || !d_n_cold)
        return HL_EINVAL;
    if (!window_ok(ctx, stage_row0, stage_rows)) return HL_EINVAL;
    if ((d_prev_cold_rows != nullptr) != (d_n_prev != nullptr) || (d_prev_cold_rows && !d_fwd_src)) return HL_EINVAL;
    return gather_impl(ctx, non, d_n_non, host_table, d_cache, stage_row0, stage_rows, d_cold_rows, d_n_cold,
                       d_prev_cold_rows, d_n_prev, d_fwd_src, static_cast<cudaEvent_t>(record_after_index),
                       static_cast<cudaEvent_t>(wait_before_move_a), static_cast<cudaEvent_t>(wait_before_move_b), true,
                       true, static_cast<cudaStream_t>(stream_));
}

extern "C" int32_t hl_index_cold(hl_ctx* ctx, hl_ubatch* non, const int32_t* d_n_non, int64_t stage_row0,
                                 int64_t stage_rows, int32_t* d_cold_rows, int64_t* d_n_cold,
                                 const int32_t* d_prev_cold_rows, const int64_t* d_n_prev, int32_t* d_fwd_src,
                                 void* stream_) {
    if (!ctx || !non || !non->offsets || !d_n_non || !d_cold_rows || !d_n_cold) return HL_EINVAL;
    if (!window_ok(ctx, stage_row0, stage_rows)) return HL_EINVAL;
    if ((d_prev_cold_rows != nullptr) != (d_n_prev != nullptr) || (d_prev_cold_rows && !d_fwd_src)) return HL_EINVAL;
    return gather_impl(ctx, non, d_n_non, nullptr, nullptr, stage_row0, stage_rows, d_cold_rows, d_n_cold,
                       d_prev_cold_rows, d_n_prev, d_fwd_src, nullptr, nullptr, nullptr, true, false,
                       static_cast<cudaStream_t>(stream_));
}

extern "C" int32_t hl_index_cold_begin(hl_ctx* ctx, hl_ubatch* non, const int32_t* d_n_non, int64_t stage_row0,
                                       int64_t stage_rows, int32_t* d_cold_rows, int64_t* d_n_cold, void* stream_) {
    if (!ctx || !non || !non->offsets || !d_n_non || !d_cold_rows || !d_n_cold) return HL_EINVAL;
    if (!window_ok(ctx, stage_row0, stage_rows)) return HL_EINVAL;
    return index_begin(ctx, non, d_n_non, stage_row0, stage_rows, d_cold_rows, d_n_cold,
                       static_cast<cudaStream_t>(stream_));
}

extern "C" const int32_t* hl_index_cold_verdict(hl_ctx* ctx) { return ctx ? ctx->r.cold_n + 1 : nullptr; }

extern "C" int32_t hl_index_cold_end(hl_ctx* ctx, hl_ubatch* non, int64_t stage_row0, int64_t stage_rows,
                                     int32_t* d_cold_rows, int64_t* d_n_cold, const int32_t* d_prev_cold_rows,
                                     const int64_t* d_n_prev, int32_t* d_fwd_src, int32_t general_not_needed,
                                     void* stream_) {
    if (!ctx || !non || !d_cold_rows || !d_n_cold) return HL_EINVAL;
    if (!window_ok(ctx, stage_row0, stage_rows)) return HL_EINVAL;
    if ((d_prev_cold_rows != nullptr) != (d_n_prev != nullptr) || (d_prev_cold_rows && !d_fwd_src)) return HL_EINVAL;
    (void)general_not_needed;
    return index_end(ctx, stage_rows, d_cold_rows, d_n_cold, d_prev_cold_rows, d_n_prev, d_fwd_src,
                     static_cast<cudaStream_t>(stream_));
}

extern "C" int32_t hl_stage_cold(hl_ctx* ctx, const float* host_table, float* d_cache, int64_t stage_row0,
                                 int64_t stage_rows, const int32_t* d_cold_rows, const int64_t* d_n_cold,
                                 const int32_t* d_fwd_src, void* stream_) {
    if (!ctx || !host_table || !d_cache || !d_cold_rows || !d_n_cold) return HL_EINVAL;
    if (!window_ok(ctx, stage_row0, stage_rows)) return HL_EINVAL;
    return gather_impl(ctx, nullptr, nullptr, host_table, d_cache, stage_row0, stage_rows,
                       const_cast<int32_t*>(d_cold_rows), const_cast<int64_t*>(d_n_cold), nullptr, nullptr,
                       const_cast<int32_t*>(d_fwd_src), nullptr, nullptr, nullptr, false, true,
                       static_cast<cudaStream_t>(stream_));
}

extern "C" int32_t hl_forward_cold(hl_ctx* ctx, float* d_cache, int64_t from_stage_row0, int64_t to_stage_row0,
                                   int64_t stage_rows, const int32_t* d_fwd_src, const int64_t* d_n_cold,
                                   void* stream_) {
    if (!ctx || !d_cache || !d_fwd_src || !d_n_cold) return HL_EINVAL;
    if (!window_ok(ctx, from_stage_row0, stage_rows) || !window_ok(ctx, to_stage_row0, stage_rows)) return HL_EINVAL;
    if (stage_rows == 0) return HL_OK;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    const int D4 = ctx->D / 4;
    const int grid = 2 * ctx_sms(ctx);
    const int64_t from = ctx->hot_cap + from_stage_row0, to = ctx->hot_cap + to_stage_row0;
    if (D4 <= 4) k_forward_rows<4><<<grid, kThreads, 0, stream>>>(d_cache, from, to, d_fwd_src, d_n_cold, stage_rows, D4);
    else if (D4 <= 8) k_forward_rows<8><<<grid, kThreads, 0, stream>>>(d_cache, from, to, d_fwd_src, d_n_cold, stage_rows, D4);
    else if (D4 <= 16) k_forward_rows<16><<<grid, kThreads, 0, stream>>>(d_cache, from, to, d_fwd_src, d_n_cold, stage_rows, D4);
    else k_forward_rows<32><<<grid, kThreads, 0, stream>>>(d_cache, from, to, d_fwd_src, d_n_cold, stage_rows, D4);
    note_launches(1);
    HL_LAUNCH_CHECK();
    return HL_OK;
}

extern "C" int32_t hl_scatter_cold_at(hl_ctx* ctx, const float* d_cache, int64_t stage_row0, int64_t stage_rows,
                                      const int32_t* d_cold_rows, const int64_t* d_n_cold, float* host_table,
                                      void* stream_) {
    if (!ctx || !d_cache || !d_cold_rows || !d_n_cold || !host_table) return HL_EINVAL;
    if (!window_ok(ctx, stage_row0, stage_rows)) return HL_EINVAL;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    timer_mark(ctx, HL_TIMER_SCATTER_MOVE, 0, stream);
    const int32_t st = launch_move_rows<true>(const_cast<float*>(d_cache), ctx->hot_cap + stage_row0,
                                              table_map(ctx, host_table),
                                              d_cold_rows, d_n_cold, stage_rows, ctx->N, ctx->D, nullptr,
                                              move_cfg(ctx, ctx->scatter_ctas), ctx->r.status, stream);
    timer_mark(ctx, HL_TIMER_SCATTER_MOVE, 1, stream);
    return st;
}

extern "C" int32_t hl_scatter_cold(hl_ctx* ctx, const float* d_cache, const int32_t* d_cold_rows,
                                   const int64_t* d_n_cold, float* host_table, void* stream_) {
    if (!ctx) return HL_EINVAL;
    return hl_scatter_cold_at(ctx, d_cache, 0, ctx->staging_cap, d_cold_rows, d_n_cold, host_table, stream_);
}

extern "C" int32_t hl_flush_hot(hl_ctx* ctx, const float* d_cache, const int32_t* d_hot_rows, const int64_t* d_n_hot,
                                float* host_table, void* stream_) {
    if (!ctx || !d_cache || !d_hot_rows || !d_n_hot || !host_table) return HL_EINVAL;
    // runs between learning phases, with nothing else on the chip: the mover at the link's full rate
    return launch_move_rows<true>(const_cast<float*>(d_cache), 0, table_map(ctx, host_table), d_hot_rows, d_n_hot,
                                  ctx->hot_cap, ctx->N,
                                  ctx->D, nullptr, move_cfg(ctx, 0), ctx->r.status, static_cast<cudaStream_t>(stream_));
}
