// Learning phase: exact access counting, selection of the popular rows, and the remap structure.
#include "hl_common.cuh"

namespace hl {
namespace {

constexpr int kThreads = 256;

// ---- counting -----------------------------------------------------------------------------------------------
// One thread per bag; a bag's table follows from its position (table-major layout).
__global__ void __launch_bounds__(kThreads) k_count(const int32_t* __restrict__ indices,
                                                    const int32_t* __restrict__ offsets, int64_t n_bags,
                                                    int64_t bags_per_table, const int64_t* __restrict__ table_base,
                                                    uint32_t* __restrict__ counts, SelectState* sel,
                                                    int32_t* status) {
    unsigned long long mine = 0;
    for (int64_t bag = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; bag < n_bags;
         bag += (int64_t)gridDim.x * blockDim.x) {
        const int t = (int)(bag / bags_per_table);
        const int64_t base = table_base[t], rows = table_base[t + 1] - base;
        const int32_t lo = offsets[bag], hi = offsets[bag + 1];
        for (int32_t j = lo; j < hi; ++j) {
            const int32_t idx = indices[j];
            if (idx < 0 || idx >= rows) {
                set_status(status, HL_EBOUNDS);
                continue;
            }
            atomicAdd(&counts[base + idx], 1u);
            ++mine;
        }
    }
#pragma unroll
    for (int d = 16; d > 0; d >>= 1) mine += __shfl_down_sync(0xffffffffu, mine, d);
    if ((threadIdx.x & 31) == 0 && mine) atomicAdd(&sel->total, mine);
}

// ---- selection: k-th largest admissible count by 8-bit radix select, most significant digit first ----------
__global__ void k_select_begin(SelectState* sel, unsigned long long k, long long share_num, long long share_den) {
    for (int i = threadIdx.x; i < 256; i += blockDim.x) sel->hist[i] = 0;
    if (threadIdx.x == 0) {
        unsigned int c_min = 1;
        if (share_num > 0) {   // count * den >= total * num  <=>  count >= ceil(total * num / den)
            const unsigned __int128 prod = (unsigned __int128)sel->total * (unsigned __int128)share_num;
            const unsigned __int128 q = (prod + (unsigned __int128)(share_den - 1)) / (unsigned __int128)share_den;
            c_min = q > 0xffffffffull ? 0xffffffffu : (unsigned int)q;
            if (c_min < 1) c_min = 1;
        }
        sel->c_min = c_min;
        sel->k_remaining = k;
        sel->prefix = 0;
        sel->mask = 0;
        sel->take_all = 0;
        sel->threshold = c_min;
        sel->quota_eq = ~0ull;
    }
}

__global__ void __launch_bounds__(kThreads) k_select_hist(const uint32_t* __restrict__ counts, int64_t N, int shift,
                                                          SelectState* sel) {
    __shared__ unsigned int h[256];
    h[threadIdx.x] = 0;
    __syncthreads();
    const unsigned int c_min = sel->c_min, prefix = sel->prefix, mask = sel->mask;
    for (int64_t g = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; g < N; g += (int64_t)gridDim.x * blockDim.x) {
        const unsigned int c = counts[g];
        if (c >= c_min && (c & mask) == prefix) atomicAdd(&h[(c >> shift) & 255u], 1u);
    }
    __syncthreads();
    if (h[threadIdx.x]) atomicAdd(&sel->hist[threadIdx.x], (unsigned long long)h[threadIdx.x]);
}

// Single thread: pick the digit that holds the k-th largest count, then clear the histogram.
__global__ void k_select_pick(SelectState* sel, int shift) {
    if (threadIdx.x == 0 && !sel->take_all) {
        unsigned long long cum = 0;
        int chosen = -1;
        for (int d = 255; d >= 0; --d) {
            const unsigned long long c = sel->hist[d];
            if (cum + c >= sel->k_remaining) {
                chosen = d;
                break;
            }
            cum += c;
        }
        if (sel->k_remaining == 0) {
            // nothing wanted: a threshold no count exceeds, and no row at the threshold either
            sel->take_all = 1;
            sel->threshold = 0xffffffffu;
            sel->quota_eq = 0ull;
        } else if (chosen < 0) {
            // fewer admissible rows than wanted: keep them all (threshold = c_min, no quota)
            sel->take_all = 1;
            sel->threshold = sel->c_min;
            sel->quota_eq = ~0ull;
        } else {
            sel->k_remaining -= cum;
            sel->prefix |= (unsigned int)chosen << shift;
            sel->mask |= 255u << shift;
            if (shift == 0) {
                sel->threshold = sel->prefix;
                sel->quota_eq = sel->k_remaining;
            }
        }
    }
    __syncthreads();
    for (int i = threadIdx.x; i < 256; i += blockDim.x) sel->hist[i] = 0;
}

__device__ __forceinline__ int warp_inclusive_scan_u(int v) {
    const int lane = threadIdx.x & 31;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
        int o = __shfl_up_sync(0xffffffffu, v, d);
        if (lane >= d) v += o;
    }
    return v;
}

// Exclusive block scan of two counters at once (256 threads).
__device__ __forceinline__ void block_scan2(int a, int b, int& ea, int& eb, int& ta, int& tb) {
    __shared__ int sa[9], sb[9];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int ia = warp_inclusive_scan_u(a), ib = warp_inclusive_scan_u(b);
    if (lane == 31) {
        sa[warp] = ia;
        sb[warp] = ib;
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        int ra = 0, rb = 0;
        for (int w = 0; w < 8; ++w) {
            const int xa = sa[w], xb = sb[w];
            sa[w] = ra;
            sb[w] = rb;
            ra += xa;
            rb += xb;
        }
        sa[8] = ra;
        sb[8] = rb;
    }
    __syncthreads();
    ea = sa[warp] + ia - a;
    eb = sb[warp] + ib - b;
    ta = sa[8];
    tb = sb[8];
    __syncthreads();
}

constexpr int kSelPer = kSelTile / kThreads;   // 16 consecutive rows per thread

__global__ void __launch_bounds__(kThreads) k_select_tile_counts(const uint32_t* __restrict__ counts, int64_t N,
                                                                 const SelectState* __restrict__ sel,
                                                                 uint32_t* __restrict__ tile_gt,
                                                                 uint32_t* __restrict__ tile_eq) {
    const unsigned int thr = sel->threshold, c_min = sel->c_min;
    const int64_t base = (int64_t)blockIdx.x * kSelTile + (int64_t)threadIdx.x * kSelPer;
    int gt = 0, eq = 0;
#pragma unroll
    for (int i = 0; i < kSelPer; ++i) {
        if (base + i < N) {
            const unsigned int c = counts[base + i];
            gt += (c > thr && c >= c_min);
            eq += (c == thr && c >= c_min);
        }
    }
    int ea, eb, ta, tb;
    block_scan2(gt, eq, ea, eb, ta, tb);
    if (threadIdx.x == 0) {
        tile_gt[blockIdx.x] = ta;
        tile_eq[blockIdx.x] = tb;
    }
}

// Single block: exclusive scans of both tile arrays in place; entry [n_tiles] = total.
__global__ void __launch_bounds__(1024) k_select_spine(uint32_t* gt, uint32_t* eq, int64_t n_tiles) {
    __shared__ unsigned int sa[33], sb[33];
    unsigned int carry_a = 0, carry_b = 0;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    for (int64_t start = 0; start < n_tiles; start += 1024) {
        const int64_t i = start + threadIdx.x;
        const unsigned int a = i < n_tiles ? gt[i] : 0, b = i < n_tiles ? eq[i] : 0;
        unsigned int ia = a, ib = b;
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
            unsigned int oa = __shfl_up_sync(0xffffffffu, ia, d), ob = __shfl_up_sync(0xffffffffu, ib, d);
            if (lane >= d) {
                ia += oa;
                ib += ob;
            }
        }
        if (lane == 31) {
            sa[warp] = ia;
            sb[warp] = ib;
        }
        __syncthreads();
        if (threadIdx.x == 0) {
            unsigned int ra = 0, rb = 0;
            for (int w = 0; w < 32; ++w) {
                const unsigned int xa = sa[w], xb = sb[w];
                sa[w] = ra;
                sb[w] = rb;
                ra += xa;
                rb += xb;
            }
            sa[32] = ra;
            sb[32] = rb;
        }
        __syncthreads();
        if (i < n_tiles) {
            gt[i] = carry_a + sa[warp] + ia - a;
            eq[i] = carry_b + sb[warp] + ib - b;
        }
        carry_a += sa[32];
        carry_b += sb[32];
        __syncthreads();
    }
    if (threadIdx.x == 0) {
        gt[n_tiles] = carry_a;
        eq[n_tiles] = carry_b;
    }
}

// Ordered compaction: a row is popular if its count beats the threshold, or equals it and fewer than quota_eq
// equal rows precede it.  Its position = popular rows with a smaller id.
__global__ void __launch_bounds__(kThreads) k_select_emit(const uint32_t* __restrict__ counts, int64_t N,
                                                          const SelectState* __restrict__ sel,
                                                          const uint32_t* __restrict__ tile_gt,
                                                          const uint32_t* __restrict__ tile_eq, int64_t n_tiles,
                                                          int64_t hot_cap, int32_t* __restrict__ hot_rows,
                                                          int64_t* __restrict__ n_hot, int32_t* status) {
    const unsigned int thr = sel->threshold, c_min = sel->c_min;
    const unsigned long long quota = sel->quota_eq;
    const int64_t base = (int64_t)blockIdx.x * kSelTile + (int64_t)threadIdx.x * kSelPer;
    unsigned int c[kSelPer];
    int gt = 0, eq = 0;
#pragma unroll
    for (int i = 0; i < kSelPer; ++i) {
        c[i] = base + i < N ? counts[base + i] : 0u;
        gt += (c[i] > thr && c[i] >= c_min);
        eq += (c[i] == thr && c[i] >= c_min);
    }
    int ea, eb, ta, tb;
    block_scan2(gt, eq, ea, eb, ta, tb);
    unsigned long long n_gt = (unsigned long long)tile_gt[blockIdx.x] + ea;
    unsigned long long n_eq = (unsigned long long)tile_eq[blockIdx.x] + eb;
#pragma unroll
    for (int i = 0; i < kSelPer; ++i) {
        if (c[i] < c_min) continue;
        const bool is_gt = c[i] > thr, is_eq = c[i] == thr;
        if (is_gt || (is_eq && n_eq < quota)) {
            const unsigned long long pos = n_gt + (n_eq < quota ? n_eq : quota);
            if ((int64_t)pos < hot_cap) hot_rows[pos] = (int32_t)(base + i);
            else set_status(status, HL_ECAPACITY);
        }
        n_gt += is_gt;
        n_eq += is_eq;
    }
    if (blockIdx.x == 0 && threadIdx.x == 0) {
        const unsigned long long all_eq = tile_eq[n_tiles];
        unsigned long long total = (unsigned long long)tile_gt[n_tiles] + (all_eq < quota ? all_eq : quota);
        if ((int64_t)total > hot_cap) total = (unsigned long long)hot_cap;
        *n_hot = (int64_t)total;
    }
}

// ---- remap --------------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(kThreads) k_remap_bits(const int32_t* __restrict__ hot_rows,
                                                         const int64_t* __restrict__ d_n_hot, int64_t hot_cap,
                                                         int64_t N, RemapBlock* remap, int32_t* status) {
    int64_t n = *d_n_hot;
    if (n > hot_cap) {
        if (blockIdx.x == 0 && threadIdx.x == 0) set_status(status, HL_ECAPACITY);
        n = hot_cap;
    }
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (int64_t)gridDim.x * blockDim.x) {
        const int64_t g = hot_rows[i];
        if (g < 0 || g >= N || (i > 0 && hot_rows[i - 1] >= g)) {   // must be strictly ascending, in range
            set_status(status, HL_EINVAL);
            continue;
        }
        const uint32_t blk = (uint32_t)(g / kRemapRowsPerBlock), r = (uint32_t)(g % kRemapRowsPerBlock);
        atomicOr(&remap[blk].w[1 + (r >> 5)], 1u << (r & 31));
    }
}

// prefix of a block = number of popular rows below its first row = lower bound in the ascending list
__global__ void __launch_bounds__(kThreads) k_remap_prefix(const int32_t* __restrict__ hot_rows,
                                                           const int64_t* __restrict__ d_n_hot, int64_t hot_cap,
                                                           int64_t n_blocks, RemapBlock* remap) {
    int64_t n = *d_n_hot;
    if (n > hot_cap) n = hot_cap;
    for (int64_t b = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; b < n_blocks;
         b += (int64_t)gridDim.x * blockDim.x) {
        const int64_t first = b * kRemapRowsPerBlock;
        int64_t lo = 0, hi = n;
        while (lo < hi) {
            const int64_t mid = (lo + hi) >> 1;
            if (hot_rows[mid] < first) lo = mid + 1;
            else hi = mid;
        }
        remap[b].w[0] = (uint32_t)lo;
    }
}

__global__ void __launch_bounds__(kThreads) k_remap_dense(const RemapBlock* __restrict__ remap, int64_t N,
                                                          int32_t* __restrict__ out) {
    for (int64_t g = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; g < N; g += (int64_t)gridDim.x * blockDim.x)
        out[g] = remap_slot(remap, g);
}

}  // namespace

// implemented in hl_cold.cu: dst[(dst_row0 + i), :] = table[rows[i], :] for i < *d_n (clamped to n_max)
int32_t launch_gather_rows(hl_ctx* ctx, float* dst, int64_t dst_row0, const float* table, const int32_t* rows,
                           const int64_t* d_n, int64_t n_max, int32_t* status, cudaStream_t stream);


// The rows [0, n) whose counts are among the k largest (count >= 1, and count * share_den >= total * share_num if
// share_num > 0; sel->total holds the total), ties at the threshold going to the smaller index; their indices, in
// ascending order, to out_idx [cap], their number to *d_n_out.  sel_gt / sel_eq: div_up(n, kSelTile) + 2 words each.
int32_t select_rows_by_count(const uint32_t* counts, int64_t n, SelectState* sel, uint32_t* sel_gt, uint32_t* sel_eq,
                             long long k, long long share_num, long long share_den, int64_t cap, int32_t* out_idx,
                             int64_t* d_n_out, int32_t* status, int sms, cudaStream_t stream) {
    const int64_t n_tiles = div_up(n, kSelTile);
    k_select_begin<<<1, 256, 0, stream>>>(sel, (unsigned long long)k, share_num, share_den);
    const int grid = grid_for(n, kThreads * 16, sms * 8);
    for (int shift = 24; shift >= 0; shift -= 8) {
        k_select_hist<<<grid, kThreads, 0, stream>>>(counts, n, shift, sel);
        k_select_pick<<<1, 256, 0, stream>>>(sel, shift);
    }
    k_select_tile_counts<<<(unsigned)n_tiles, kThreads, 0, stream>>>(counts, n, sel, sel_gt, sel_eq);
    k_select_spine<<<1, 1024, 0, stream>>>(sel_gt, sel_eq, n_tiles);
    k_select_emit<<<(unsigned)n_tiles, kThreads, 0, stream>>>(counts, n, sel, sel_gt, sel_eq, n_tiles, cap, out_idx,
                                                             d_n_out, status);
    note_launches(12);   // begin, 4 x (histogram, pick), tile counts, spine, emit
    HL_LAUNCH_CHECK();
    return HL_OK;
}

}  // namespace hl

using namespace hl;

extern "C" int32_t hl_profile_hot(hl_ctx* ctx, const hl_batch* b, int32_t reset, int32_t finalize, int32_t policy,
                                  int64_t p_num, int64_t p_den, int32_t* d_hot_rows, int64_t* d_n_hot,
                                  void* stream_) {
    if (!ctx) return HL_EINVAL;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    Regions& r = ctx->r;
    if (reset) {
        HL_CUDA_TRY(cudaMemsetAsync(r.counts, 0, sizeof(uint32_t) * ctx->N, stream));
        HL_CUDA_TRY(cudaMemsetAsync(r.sel, 0, sizeof(SelectState), stream));
    }
    if (b) {
        if (b->batch < 1 || b->batch > ctx->max_batch || b->nnz < 0 || b->nnz > ctx->max_nnz || !b->offsets ||
            (b->nnz > 0 && !b->indices))
            return HL_EINVAL;
        const int64_t bags_per_table = (int64_t)b->batch * ctx->S;
        const int64_t n_bags = bags_per_table * ctx->T;
        k_count<<<grid_for(n_bags, kThreads, ctx_sms(ctx) * 8), kThreads, 0, stream>>>(
            b->indices, b->offsets, n_bags, bags_per_table, r.table_base, r.counts, r.sel, r.status);
        note_launches(1);
        HL_LAUNCH_CHECK();
    }
    if (finalize) {
        if (!d_hot_rows || !d_n_hot) return HL_EINVAL;
        long long k = 0, share_num = 0, share_den = 1;
        switch (policy) {
            case HL_HOT_TOPK_ROWS: k = p_num; break;
            case HL_HOT_BUDGET_BYTES: k = p_num / (4 * (int64_t)ctx->D); break;
            case HL_HOT_FRACTION_ROWS:
                if (p_den <= 0 || p_num < 0) return HL_EINVAL;
                k = (long long)(((__int128)ctx->N * p_num) / p_den);
                break;
            case HL_HOT_MIN_SHARE:
                if (p_den <= 0 || p_num <= 0) return HL_EINVAL;
                k = ctx->hot_cap;
                share_num = p_num;
                share_den = p_den;
                break;
            default: return HL_EINVAL;
        }
        if (k < 0) return HL_EINVAL;
        if (k > ctx->hot_cap) k = ctx->hot_cap;
        return select_rows_by_count(r.counts, ctx->N, r.sel, r.sel_gt, r.sel_eq, k, share_num, share_den, ctx->hot_cap,
                                    d_hot_rows, d_n_hot, r.status, ctx_sms(ctx), stream);
    }
    return HL_OK;
}

extern "C" int32_t hl_build_remap(hl_ctx* ctx, const int32_t* d_hot_rows, const int64_t* d_n_hot,
                                  const float* host_table, float* d_cache, int32_t* d_remap_out, void* stream_) {
    if (!ctx || !d_hot_rows || !d_n_hot) return HL_EINVAL;
    if (host_table && !d_cache) return HL_EINVAL;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    Regions& r = ctx->r;
    HL_CUDA_TRY(cudaMemsetAsync(r.remap, 0, sizeof(RemapBlock) * ctx->n_remap_blocks, stream));
    if (ctx->hot_cap > 0) {
        k_remap_bits<<<grid_for(ctx->hot_cap, kThreads, ctx_sms(ctx) * 8), kThreads, 0, stream>>>(
            d_hot_rows, d_n_hot, ctx->hot_cap, ctx->N, r.remap, r.status);
        note_launches(1);
    }
    k_remap_prefix<<<grid_for(ctx->n_remap_blocks, kThreads, ctx_sms(ctx) * 8), kThreads, 0, stream>>>(
        d_hot_rows, d_n_hot, ctx->hot_cap, ctx->n_remap_blocks, r.remap);
    note_launches(d_remap_out ? 2 : 1);
    if (d_remap_out)
        k_remap_dense<<<grid_for(ctx->N, kThreads * 4, ctx_sms(ctx) * 16), kThreads, 0, stream>>>(r.remap, ctx->N,
                                                                                         d_remap_out);
    HL_LAUNCH_CHECK();
    if (host_table && ctx->hot_cap > 0)
        return launch_gather_rows(ctx, d_cache, 0, host_table, d_hot_rows, d_n_hot, ctx->hot_cap, r.status, stream);
    return HL_OK;
}
