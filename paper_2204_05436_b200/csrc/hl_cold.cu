// The non-popular micro-batch's working set: classify its lookups, find the distinct cold rows, stage them from
// the host-DRAM table (zero-copy 128-bit loads over the host link) behind the hot cache, and write them back.
#include "hl_common.cuh"

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

__global__ void __launch_bounds__(kThreads) k_cold_heads(const int32_t* __restrict__ keys,
                                                         const int32_t* __restrict__ d_n, int64_t n_max,
                                                         int32_t* __restrict__ heads) {
    int64_t n = *d_n;
    n = n < n_max ? n : n_max;
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (int64_t)gridDim.x * blockDim.x)
        heads[i] = (i == 0 || keys[i] != keys[i - 1]) ? 1 : 0;
}

// rank_excl[i] = number of run heads before i; the row at i has rank rank_excl[i] if it is a head, else
// rank_excl[i] - 1.
__global__ void __launch_bounds__(kThreads) k_cold_assign(const int32_t* __restrict__ keys,
                                                          const int32_t* __restrict__ vals,
                                                          const int32_t* __restrict__ d_n, int64_t n_max,
                                                          const int32_t* __restrict__ rank_excl, int64_t hot_cap,
                                                          int64_t staging_cap, int32_t* __restrict__ ids,
                                                          int32_t* __restrict__ cold_rows,
                                                          int64_t* __restrict__ d_n_cold, int32_t* status) {
    int64_t n = *d_n;
    n = n < n_max ? n : n_max;
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
        if (rank < staging_cap) {
            if (head) cold_rows[rank] = keys[i];
            ids[vals[i]] = (int32_t)(hot_cap + rank);
        } else {
            ids[vals[i]] = -1;   // no room to stage this row: the lookup is dropped and the status word says so
        }
    }
}

// dst[(dst_row0 + i), :] = table[rows[i], :]; G lanes per row, UR rows in flight per group.
template <int G, bool TO_TABLE>
__global__ void __launch_bounds__(kThreads) k_move_rows(float* __restrict__ dense_side, int64_t dense_row0,
                                                        float* __restrict__ table, const int32_t* __restrict__ rows,
                                                        const int64_t* __restrict__ d_n, int64_t n_max,
                                                        int64_t table_rows, int D4, int32_t* status) {
    constexpr int UR = 4;
    int64_t n = *d_n;
    n = n < 0 ? 0 : (n < n_max ? n : n_max);
    const int sub = threadIdx.x % G;
    const int64_t group = ((int64_t)blockIdx.x * kThreads + threadIdx.x) / G;
    const int64_t n_groups = (int64_t)gridDim.x * kThreads / G;
    float4* dense4 = reinterpret_cast<float4*>(dense_side) + dense_row0 * D4;
    float4* table4 = reinterpret_cast<float4*>(table);
    for (int64_t i0 = group * UR; i0 < n; i0 += n_groups * UR) {
        int64_t g[UR];
#pragma unroll
        for (int u = 0; u < UR; ++u) {
            g[u] = i0 + u < n ? (int64_t)rows[i0 + u] : -1;
            if (g[u] >= table_rows) {
                set_status(status, HL_EBOUNDS);
                g[u] = -1;
            }
        }
        for (int c = sub; c < D4; c += G) {
            float4 v[UR];
#pragma unroll
            for (int u = 0; u < UR; ++u)
                if (g[u] >= 0) v[u] = TO_TABLE ? dense4[(i0 + u) * D4 + c] : table4[g[u] * D4 + c];
#pragma unroll
            for (int u = 0; u < UR; ++u)
                if (g[u] >= 0) {
                    if (TO_TABLE) table4[g[u] * D4 + c] = v[u];
                    else dense4[(i0 + u) * D4 + c] = v[u];
                }
        }
    }
}

template <bool TO_TABLE>
int32_t launch_move_rows(float* dense_side, int64_t dense_row0, float* table, const int32_t* rows,
                         const int64_t* d_n, int64_t n_max, int64_t table_rows, int D, int32_t* status,
                         cudaStream_t stream) {
    if (n_max <= 0) return HL_OK;
    const int D4 = D / 4;
    // Two light CTAs per SM: random rows of a table of tens of GB miss the address translation of the host
    // link on almost every row, and the link only reaches its rate with many such misses in flight at once
    // (measured: 32 CTAs 19 GB/s, 296 and more 24 GB/s on random rows; 50 GB/s on rows within 4 GB either way).
    const int grid = 2 * kSMs;
    if (D4 <= 4)
        k_move_rows<4, TO_TABLE><<<grid, kThreads, 0, stream>>>(dense_side, dense_row0, table, rows, d_n, n_max,
                                                               table_rows, D4, status);
    else if (D4 <= 8)
        k_move_rows<8, TO_TABLE><<<grid, kThreads, 0, stream>>>(dense_side, dense_row0, table, rows, d_n, n_max,
                                                               table_rows, D4, status);
    else if (D4 <= 16)
        k_move_rows<16, TO_TABLE><<<grid, kThreads, 0, stream>>>(dense_side, dense_row0, table, rows, d_n, n_max,
                                                                table_rows, D4, status);
    else
        k_move_rows<32, TO_TABLE><<<grid, kThreads, 0, stream>>>(dense_side, dense_row0, table, rows, d_n, n_max,
                                                                table_rows, D4, status);
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

int32_t launch_gather_rows(float* dst, int64_t dst_row0, const float* table, const int32_t* rows,
                           const int64_t* d_n, int64_t n_max, int64_t table_rows, int D, int32_t* status,
                           cudaStream_t stream) {
    return launch_move_rows<false>(dst, dst_row0, const_cast<float*>(table), rows, d_n, n_max, table_rows, D, status,
                                   stream);
}

}  // namespace hl

using namespace hl;

extern "C" int32_t hl_gather_cold(hl_ctx* ctx, hl_ubatch* non, const int32_t* d_n_non, const float* host_table,
                                  float* d_cache, int32_t* d_cold_rows, int64_t* d_n_cold, void* stream_) {
    if (!ctx || !non || !non->offsets || !d_n_non || !host_table || !d_cache || !d_cold_rows || !d_n_cold)
        return HL_EINVAL;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    Regions& r = ctx->r;
    if (ctx->max_nnz == 0) {
        HL_CUDA_TRY(cudaMemsetAsync(d_n_cold, 0, sizeof(int64_t), stream));
        return HL_OK;
    }
    if (!non->ids) return HL_EINVAL;
    HL_CUDA_TRY(cudaMemsetAsync(r.cold_n, 0, 4 * sizeof(int32_t), stream));
    const int grid = grid_for(ctx->max_nnz, kThreads, kSMs * 4);
    k_cold_classify<<<grid, kThreads, 0, stream>>>(non->ids, non->offsets, d_n_non, ctx->max_batch, ctx->T * ctx->S,
                                                   non->cap_ids, ctx->N, r.remap, r.cold_keys[0], r.cold_vals[0],
                                                   r.cold_n, ctx->max_nnz, r.status);
    note_launches(1);
    HL_LAUNCH_CHECK();
    int32_t *keys, *vals;
    int32_t st = radix_sort_pairs(r.cold_keys, r.cold_vals, r.cold_n, ctx->max_nnz, bits_for(ctx->N - 1),
                                  r.cold_hist, r.status, &keys, &vals, stream);
    if (st != HL_OK) return st;
    k_cold_heads<<<grid, kThreads, 0, stream>>>(keys, r.cold_n, ctx->max_nnz, r.cold_rank);
    note_launches(1);
    HL_LAUNCH_CHECK();
    st = exclusive_scan_i32(r.cold_rank, r.cold_rank, r.cold_n, ctx->max_nnz, r.cold_tiles, r.status, stream);
    if (st != HL_OK) return st;
    k_cold_assign<<<grid, kThreads, 0, stream>>>(keys, vals, r.cold_n, ctx->max_nnz, r.cold_rank, ctx->hot_cap,
                                                 ctx->staging_cap, non->ids, d_cold_rows, d_n_cold, r.status);
    note_launches(1);
    HL_LAUNCH_CHECK();
    timer_mark(ctx, HL_TIMER_GATHER_MOVE, 0, stream);
    st = launch_move_rows<false>(d_cache, ctx->hot_cap, const_cast<float*>(host_table), d_cold_rows, d_n_cold,
                                 ctx->staging_cap, ctx->N, ctx->D, r.status, stream);
    timer_mark(ctx, HL_TIMER_GATHER_MOVE, 1, stream);
    return st;
}

extern "C" int32_t hl_scatter_cold(hl_ctx* ctx, const float* d_cache, const int32_t* d_cold_rows,
                                   const int64_t* d_n_cold, float* host_table, void* stream_) {
    if (!ctx || !d_cache || !d_cold_rows || !d_n_cold || !host_table) return HL_EINVAL;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    timer_mark(ctx, HL_TIMER_SCATTER_MOVE, 0, stream);
    const int32_t st = launch_move_rows<true>(const_cast<float*>(d_cache), ctx->hot_cap, host_table, d_cold_rows,
                                              d_n_cold, ctx->staging_cap, ctx->N, ctx->D, ctx->r.status, stream);
    timer_mark(ctx, HL_TIMER_SCATTER_MOVE, 1, stream);
    return st;
}
