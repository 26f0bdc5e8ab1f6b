// The approximate access logger of the learning phase (Section V-B "Efficient Embedding Tracking"): a set-associative
// table of row tags with a 2-bit re-reference prediction value per block, replaced by SRRIP with insertion one below
// the maximum, the set chosen by a Feistel randomizer of the (index, table) tuple (Section V-C).
//
// The ASIC serves one access after the other; the result depends on that order only within a set.  So the lookups of
// a mini-batch are keyed by their set and sorted stably (their order within a set stays the order of the layout),
// and a warp replays each set's run of the sorted list in turn, the ways of the set held one per lane.
#include "hl_common.cuh"

namespace hl {
namespace {

constexpr int kThreads = 256;
constexpr int kRrpvMax = 3;        // 2-bit counter; also the value of an empty way
constexpr int kRrpvInsert = 2;     // one below the maximum

// Four Feistel rounds on the 16-bit halves of the key; round function = upper half of (x * odd constant + round key).
__device__ __forceinline__ uint32_t randomizer(uint32_t g) {
    uint32_t left = g >> 16, right = g & 0xffffu;
    const uint32_t rk[4] = {0x85EBCA6Bu, 0xC2B2AE35u, 0x27D4EB2Fu, 0x165667B1u};
#pragma unroll
    for (int r = 0; r < 4; ++r) {
        const uint32_t f = (right * 0x9E3779B1u + rk[r]) >> 16;
        const uint32_t t = left ^ f;
        left = right;
        right = t;
    }
    return (left << 16) | right;
}

// (set, row) of every lookup, at the lookup's own position; lookups outside their table get the sentinel set n_sets.
__global__ void __launch_bounds__(kThreads) k_trk_keys(const int32_t* __restrict__ indices,
                                                       const int32_t* __restrict__ offsets, int64_t n_bags,
                                                       int64_t bags_per_table, const int64_t* __restrict__ table_base,
                                                       int64_t max_nnz, uint32_t n_sets, int32_t* __restrict__ keys,
                                                       int32_t* __restrict__ vals, int32_t* __restrict__ d_n,
                                                       int32_t* status) {
    if (blockIdx.x == 0 && threadIdx.x == 0) {
        int64_t L = offsets[n_bags];
        if (L > max_nnz) {
            set_status(status, HL_ECAPACITY);
            L = max_nnz;
        }
        d_n[0] = (int32_t)(L < 0 ? 0 : L);
    }
    for (int64_t bag = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; bag < n_bags;
         bag += (int64_t)gridDim.x * blockDim.x) {
        const int t = (int)(bag / bags_per_table);
        const int64_t base = table_base[t], rows = table_base[t + 1] - base;
        const int64_t lo = offsets[bag], hi = offsets[bag + 1];
        for (int64_t j = lo; j < hi && j < max_nnz; ++j) {
            const int32_t idx = indices[j];
            if (idx < 0 || idx >= rows) {
                set_status(status, HL_EBOUNDS);
                keys[j] = (int32_t)n_sets;
                vals[j] = -1;
            } else {
                const uint32_t g = (uint32_t)(base + idx);
                keys[j] = (int32_t)(randomizer(g) % n_sets);
                vals[j] = (int32_t)g;
            }
        }
    }
}

// One warp per 32 positions of the sorted list: every position where a new set's run begins is a head, and the warp
// replays, head after head, the accesses of that set (the run may reach far beyond the warp's own 32 positions; the
// warps there find no head in it and leave it alone).  While a set is replayed lane w holds its way w.
__global__ void __launch_bounds__(kThreads) k_trk_replay(const int32_t* __restrict__ keys,
                                                         const int32_t* __restrict__ vals,
                                                         const int32_t* __restrict__ d_n, int64_t n_max,
                                                         int32_t* __restrict__ tags, uint8_t* __restrict__ rrpv,
                                                         int64_t n_sets, int ways,
                                                         unsigned long long* __restrict__ d_hits) {
    int64_t n = d_n[0];
    n = n < 0 ? 0 : (n < n_max ? n : n_max);
    const int lane = threadIdx.x & 31;
    const int64_t n_warps = (int64_t)gridDim.x * (blockDim.x >> 5);
    unsigned long long hits = 0;
    for (int64_t w0 = ((int64_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5)) * 32; w0 < n; w0 += n_warps * 32) {
        const int64_t p = w0 + lane;
        const int32_t kp = p < n ? keys[p] : -1;
        const int32_t kprev = (p > 0 && p < n) ? keys[p - 1] : -1;
        unsigned heads = __ballot_sync(0xffffffffu, p < n && kp >= 0 && kp < n_sets && kp != kprev);
        while (heads) {
            const int h = __ffs(heads) - 1;
            heads &= heads - 1;
            const int64_t s = __shfl_sync(0xffffffffu, kp, h);
            int32_t tag = lane < ways ? tags[s * ways + lane] : -2;          // -2: matches no row
            int rr = lane < ways ? (int)rrpv[s * ways + lane] : -1;          // -1: never a victim, never aged
            int32_t last = -1;            // the row of the previous access
            bool last_zero = false;       // ... which left that row at RRPV 0, so that repeating it changes nothing
            for (int64_t i = w0 + h;; i += 32) {
                const bool in = i + lane < n;
                const int32_t k = in ? keys[i + lane] : -1;
                const int32_t g = in ? vals[i + lane] : -1;
                const int cnt = __ffs(~__ballot_sync(0xffffffffu, k == (int32_t)s)) - 1;   // leading lanes of the run
                const int c = cnt < 0 ? 32 : cnt;
                if (last_zero && __all_sync(0xffffffffu, lane >= c || g == last)) {
                    hits += c;                                                    // a burst of one popular row
                } else {
                    for (int t = 0; t < c; ++t) {
                        const int32_t gg = __shfl_sync(0xffffffffu, g, t);
                        if (gg == last && last_zero) {
                            ++hits;
                            continue;
                        }
                        const unsigned hit = __ballot_sync(0xffffffffu, tag == gg);
                        if (hit) {
                            if (lane == __ffs(hit) - 1) rr = 0;
                            last_zero = true;
                            ++hits;
                        } else {
                            unsigned vm = __ballot_sync(0xffffffffu, rr == kRrpvMax);
                            if (!vm) {   // age the whole set until its oldest block reaches the maximum
                                const int add = __ballot_sync(0xffffffffu, rr == 2) ? 1
                                                : __ballot_sync(0xffffffffu, rr == 1) ? 2 : 3;
                                if (lane < ways) rr += add;
                                vm = __ballot_sync(0xffffffffu, rr == kRrpvMax);
                            }
                            if (lane == __ffs(vm) - 1) {
                                tag = gg;
                                rr = kRrpvInsert;
                            }
                            last_zero = false;
                        }
                        last = gg;
                    }
                }
                if (c < 32) break;
            }
            if (lane < ways) {
                tags[s * ways + lane] = tag;
                rrpv[s * ways + lane] = (uint8_t)rr;
            }
        }
    }
    if (lane == 0 && d_hits && hits) atomicAdd(d_hits, hits);
}

// counts[row] = 4 - RRPV for every tracked row (the counters were cleared before).
__global__ void __launch_bounds__(kThreads) k_trk_export(const int32_t* __restrict__ tags,
                                                         const uint8_t* __restrict__ rrpv, int64_t n_blocks, int64_t N,
                                                         uint32_t* __restrict__ counts, SelectState* sel,
                                                         int32_t* status) {
    unsigned long long mine = 0;
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n_blocks;
         i += (int64_t)gridDim.x * blockDim.x) {
        const int32_t g = tags[i];
        if (g < 0) continue;
        if (g >= N || rrpv[i] > kRrpvMax) {
            set_status(status, HL_EBOUNDS);
            continue;
        }
        const uint32_t c = (uint32_t)(kRrpvMax + 1 - rrpv[i]);
        counts[g] = c;
        mine += c;
    }
#pragma unroll
    for (int d = 16; d > 0; d >>= 1) mine += __shfl_down_sync(0xffffffffu, mine, d);
    if ((threadIdx.x & 31) == 0 && mine) atomicAdd(&sel->total, mine);
}

int bits_for(int64_t max_value) {
    int b = 1;
    while ((int64_t(1) << b) <= max_value) ++b;
    return b;
}

bool tracker_shape_ok(int64_t n_sets, int32_t ways) {
    return n_sets >= 1 && n_sets < (int64_t(1) << 30) && ways >= 1 && ways <= 32;
}

}  // namespace
}  // namespace hl

using namespace hl;

extern "C" int32_t hl_tracker_reset(hl_ctx* ctx, int32_t* d_tags, uint8_t* d_rrpv, int64_t n_sets, int32_t ways,
                                    unsigned long long* d_hits, void* stream_) {
    if (!ctx || !d_tags || !d_rrpv || !tracker_shape_ok(n_sets, ways)) return HL_EINVAL;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    HL_CUDA_TRY(cudaMemsetAsync(d_tags, 0xff, sizeof(int32_t) * n_sets * ways, stream));
    HL_CUDA_TRY(cudaMemsetAsync(d_rrpv, kRrpvMax, (size_t)n_sets * ways, stream));
    if (d_hits) HL_CUDA_TRY(cudaMemsetAsync(d_hits, 0, sizeof(unsigned long long), stream));
    return HL_OK;
}

extern "C" int32_t hl_tracker_update(hl_ctx* ctx, const hl_batch* b, int32_t* d_tags, uint8_t* d_rrpv, int64_t n_sets,
                                     int32_t ways, unsigned long long* d_hits, void* stream_) {
    if (!ctx || !b || !d_tags || !d_rrpv || !tracker_shape_ok(n_sets, ways)) return HL_EINVAL;
    if (b->batch < 1 || b->batch > ctx->max_batch || b->nnz < 0 || b->nnz > ctx->max_nnz || !b->offsets ||
        (b->nnz > 0 && !b->indices))
        return HL_EINVAL;
    if (b->nnz == 0 || ctx->max_nnz == 0) return HL_OK;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    Regions& r = ctx->r;
    const int64_t bags_per_table = (int64_t)b->batch * ctx->S;
    const int64_t n_bags = bags_per_table * ctx->T;
    k_trk_keys<<<grid_for(n_bags, kThreads, kMaxGrid), kThreads, 0, stream>>>(
        b->indices, b->offsets, n_bags, bags_per_table, r.table_base, ctx->max_nnz, (uint32_t)n_sets, r.bwd_keys[0],
        r.bwd_vals[0], r.bwd_n, r.status);
    note_launches(1);
    HL_LAUNCH_CHECK();
    int32_t *keys, *vals;
    const int32_t st = radix_sort_pairs(r.bwd_keys, r.bwd_vals, r.bwd_n, ctx->max_nnz, bits_for(n_sets), r.bwd_hist,
                                        r.status, &keys, &vals, stream);
    if (st != HL_OK) return st;
    k_trk_replay<<<grid_for(ctx->max_nnz, kThreads, kMaxGrid), kThreads, 0, stream>>>(keys, vals, r.bwd_n, ctx->max_nnz,
                                                                                    d_tags, d_rrpv, n_sets, ways,
                                                                                    d_hits);
    note_launches(1);
    HL_LAUNCH_CHECK();
    return HL_OK;
}

extern "C" int32_t hl_tracker_export(hl_ctx* ctx, const int32_t* d_tags, const uint8_t* d_rrpv, int64_t n_sets,
                                     int32_t ways, void* stream_) {
    if (!ctx || !d_tags || !d_rrpv || !tracker_shape_ok(n_sets, ways)) return HL_EINVAL;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    Regions& r = ctx->r;
    HL_CUDA_TRY(cudaMemsetAsync(r.counts, 0, sizeof(uint32_t) * ctx->N, stream));
    HL_CUDA_TRY(cudaMemsetAsync(r.sel, 0, sizeof(SelectState), stream));
    const int64_t n_blocks = n_sets * ways;
    k_trk_export<<<grid_for(n_blocks, kThreads, kMaxGrid), kThreads, 0, stream>>>(d_tags, d_rrpv, n_blocks, ctx->N,
                                                                                 r.counts, r.sel, r.status);
    note_launches(1);
    HL_LAUNCH_CHECK();
    return HL_OK;
}
