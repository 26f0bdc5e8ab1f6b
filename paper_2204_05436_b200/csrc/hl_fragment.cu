// Fragmenting a mini-batch into the popular micro-batch O and the non-popular micro-batch X.
//
//   1. k_frag_flags     one warp per input: probe the popular-row bitmap for every lookup of the input,
//                       all-hit decided by a warp vote; the last CTA to finish then partitions: ballot + prefix
//                       sums over the flags -> stable partition `perm`, n_pop
//   2. k_frag_sizes     size of every destination bag (O's bags, then X's bags), then an exclusive scan
//   3. k_frag_emit      copy every bag's lookups to its place, mapped to a cache slot (O) or global row (X), and
//                       every input's dense features to its place
#include "hl_common.cuh"

namespace hl {
namespace {

constexpr int kThreads = 256;
constexpr int kFlagThreads = 1024;      // CTAs of the flags kernel: its last CTA partitions all inputs by itself

// LANE_PER_TABLE: lane l walks the lookups of tables l, l+32, ... of its input (short bags: pooling 1).
// otherwise the warp walks table after table with the lanes striding over the table's lookups of the input
// (its S bags are contiguous in the table-major layout).
// Probe: how a global row is looked up in the popular set (BitmapProbe: the dense bitmap of the 32-bit path;
// HashProbe: the hashed remap of the wide-id path).
__device__ void partition_by_flags(const uint8_t* flags, int B, int32_t* __restrict__ perm,
                                   int32_t* __restrict__ counts);

template <bool LANE_PER_TABLE, class Probe>
__global__ void __launch_bounds__(kFlagThreads) k_frag_flags(const int32_t* __restrict__ indices,
                                                         const int32_t* __restrict__ offsets, int B, int T, int S,
                                                         const int64_t* __restrict__ table_base, Probe remap,
                                                         uint8_t* flags, int32_t* status, int32_t* __restrict__ perm,
                                                         int32_t* __restrict__ counts, unsigned int* finished) {
    __shared__ bool s_last;
    const int lane = threadIdx.x & 31;
    const int warps_per_block = kFlagThreads / 32;
    for (int b = blockIdx.x * warps_per_block + (threadIdx.x >> 5); b < B; b += gridDim.x * warps_per_block) {
        bool miss = false;
        if (LANE_PER_TABLE) {
            for (int t = lane; t < T; t += 32) {
                const int64_t first_bag = ((int64_t)t * B + b) * S;
                const int32_t lo = offsets[first_bag], hi = offsets[first_bag + S];
                const int64_t base = table_base[t], rows = table_base[t + 1] - base;
                for (int32_t j = lo; j < hi; ++j) {
                    const int32_t idx = indices[j];
                    if (idx < 0 || idx >= rows) {
                        set_status(status, HL_EBOUNDS);
                        miss = true;
                    } else if (!remap.hit(base + idx)) {
                        miss = true;
                    }
                }
            }
        } else {
            for (int t = 0; t < T; ++t) {
                const int64_t first_bag = ((int64_t)t * B + b) * S;
                const int32_t lo = offsets[first_bag], hi = offsets[first_bag + S];
                const int64_t base = table_base[t], rows = table_base[t + 1] - base;
                for (int32_t j = lo + lane; j < hi; j += 32) {
                    const int32_t idx = indices[j];
                    if (idx < 0 || idx >= rows) {
                        set_status(status, HL_EBOUNDS);
                        miss = true;
                    } else if (!remap.hit(base + idx)) {
                        miss = true;
                    }
                }
            }
        }
        const unsigned any_miss = __ballot_sync(0xffffffffu, miss);
        if (lane == 0) flags[b] = any_miss == 0;
    }
    // The CTA that finishes last partitions the inputs (a launch of its own for one block's work costs more than the
    // work): every CTA's flags are written and fenced before it counts itself in, and the last one reads them past
    // its first-level cache.  The tally goes back to zero for the next call.
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0) s_last = atomicAdd(finished, 1u) == gridDim.x - 1;
    __syncthreads();
    if (!s_last) return;
    __threadfence();
    partition_by_flags(flags, B, perm, counts);
    if (threadIdx.x == 0) *finished = 0;
}

// One block.  Pass 1 counts the popular inputs; pass 2 places every input: a popular one at its rank among the
// popular, a non-popular one behind all popular ones at its rank among the non-popular.
__device__ void partition_by_flags(const uint8_t* flags, int B, int32_t* __restrict__ perm,
                                   int32_t* __restrict__ counts) {
    constexpr int NT = kFlagThreads;
    __shared__ int warp_sum[32];
    __shared__ int s_total;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const unsigned lt = lanemask_lt();
    if (threadIdx.x < 32) warp_sum[threadIdx.x] = 0;          // (fewer than 32 warps write theirs)
    __syncthreads();

    int mine = 0;
    for (int b = threadIdx.x; b < B; b += NT) mine += __ldcg(&flags[b]);
#pragma unroll
    for (int d = 16; d > 0; d >>= 1) mine += __shfl_down_sync(0xffffffffu, mine, d);
    if (lane == 0) warp_sum[warp] = mine;
    __syncthreads();
    if (threadIdx.x == 0) {
        int s = 0;
        for (int w = 0; w < 32; ++w) s += warp_sum[w];
        s_total = s;
    }
    __syncthreads();
    const int n_pop = s_total;
    __syncthreads();

    int before = 0;   // popular inputs in earlier chunks
    for (int start = 0; start < B; start += NT) {
        const int b = start + threadIdx.x;
        const bool valid = b < B;
        const bool pop = valid && __ldcg(&flags[b]);
        const unsigned vote = __ballot_sync(0xffffffffu, pop);
        if (lane == 0) warp_sum[warp] = __popc(vote);
        __syncthreads();
        if (warp == 0) {
            const int c = lane < NT / 32 ? warp_sum[lane] : 0;
            int incl = c;
#pragma unroll
            for (int d = 1; d < 32; d <<= 1) {
                int o = __shfl_up_sync(0xffffffffu, incl, d);
                if (lane >= d) incl += o;
            }
            warp_sum[lane] = incl - c;
            if (lane == 31) s_total = incl;
        }
        __syncthreads();
        if (valid) {
            const int rank_pop = before + warp_sum[warp] + __popc(vote & lt);   // popular inputs before b
            if (pop) perm[rank_pop] = b;
            else perm[n_pop + (b - rank_pop)] = b;
        }
        before += s_total;
        __syncthreads();
    }
    if (threadIdx.x == 0) {
        counts[0] = n_pop;
        counts[1] = B - n_pop;
    }
}

struct DestBag {
    int64_t src_bag;
    int t;
    bool is_pop;
};

// Destination bags: O's T*l*S bags, then X's T*k*S bags, each table-major over the micro-batch's inputs.
__device__ __forceinline__ DestBag decode_dest_bag(int64_t dst, int B, int S, int n_pop, int64_t pop_bags,
                                                   const int32_t* __restrict__ perm) {
    DestBag d;
    d.is_pop = dst < pop_bags;
    const int64_t local = d.is_pop ? dst : dst - pop_bags;
    const int n = d.is_pop ? n_pop : B - n_pop;
    const int64_t per_table = (int64_t)n * S;
    d.t = (int)(local / per_table);
    const int64_t rem = local - (int64_t)d.t * per_table;
    const int i = (int)(rem / S), s = (int)(rem - (int64_t)i * S);
    const int b = perm[(d.is_pop ? 0 : n_pop) + i];
    d.src_bag = ((int64_t)d.t * B + b) * S + s;
    return d;
}

__global__ void __launch_bounds__(kThreads) k_frag_sizes(const int32_t* __restrict__ offsets, int B, int T, int S,
                                                         const int32_t* __restrict__ perm,
                                                         const int32_t* __restrict__ counts,
                                                         int32_t* __restrict__ sizes) {
    const int n_pop = counts[0];
    const int64_t n_bags = (int64_t)T * B * S, pop_bags = (int64_t)T * n_pop * S;
    for (int64_t dst = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; dst < n_bags;
         dst += (int64_t)gridDim.x * blockDim.x) {
        const DestBag d = decode_dest_bag(dst, B, S, n_pop, pop_bags, perm);
        sizes[dst] = offsets[d.src_bag + 1] - offsets[d.src_bag];
    }
}

// GROUP lanes cooperate on one destination bag (1 for short bags, 32 for long ones).  NonId: type of X's global row
// ids (int32_t, or int64_t on the wide-id path).
template <int GROUP, class Probe, typename NonId>
__global__ void __launch_bounds__(kThreads) k_frag_emit(const int32_t* __restrict__ indices,
                                                        const int32_t* __restrict__ offsets, int B, int T, int S,
                                                        const int32_t* __restrict__ perm,
                                                        int32_t* __restrict__ counts,
                                                        const int32_t* __restrict__ dst_start,   // scanned sizes
                                                        const int64_t* __restrict__ table_base, Probe remap,
                                                        int32_t* __restrict__ pop_offsets, int32_t* __restrict__ pop_ids,
                                                        int64_t pop_cap, int32_t* __restrict__ non_offsets,
                                                        NonId* __restrict__ non_ids, int64_t non_cap,
                                                        int32_t* status, const float* __restrict__ dense,
                                                        int n_dense, float* __restrict__ dense_out) {
    const int n_pop = counts[0];
    const int64_t n_bags = (int64_t)T * B * S, pop_bags = (int64_t)T * n_pop * S;
    const int32_t L_pop = dst_start[pop_bags], L_all = dst_start[n_bags];
    const int sub = threadIdx.x % GROUP;
    const int64_t group = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) / GROUP;
    const int64_t n_groups = (int64_t)gridDim.x * blockDim.x / GROUP;
    if (group == 0 && sub == 0) {
        counts[2] = L_pop;
        counts[3] = L_all - L_pop;
        pop_offsets[pop_bags] = L_pop;
        non_offsets[n_bags - pop_bags] = L_all - L_pop;
    }
    for (int64_t dst = group; dst < n_bags; dst += n_groups) {
        const DestBag d = decode_dest_bag(dst, B, S, n_pop, pop_bags, perm);
        const int32_t src_lo = offsets[d.src_bag], src_hi = offsets[d.src_bag + 1];
        const int64_t base = table_base[d.t], rows = table_base[d.t + 1] - base;
        if (d.is_pop) {
            const int32_t out_lo = dst_start[dst];
            if (sub == 0) pop_offsets[dst] = out_lo;
            for (int32_t j = sub; j < src_hi - src_lo; j += GROUP) {
                if (out_lo + j >= pop_cap) {
                    set_status(status, HL_ECAPACITY);
                    break;
                }
                const int32_t idx = indices[src_lo + j];
                // every lookup of a popular input was tested to be in range and popular
                pop_ids[out_lo + j] = remap.slot(base + idx);
            }
        } else {
            const int32_t out_lo = dst_start[dst] - L_pop;
            if (out_lo < 0) continue;   // only after a chain poll of the scan gave up (HL_ETIMEOUT)
            if (sub == 0) non_offsets[dst - pop_bags] = out_lo;
            for (int32_t j = sub; j < src_hi - src_lo; j += GROUP) {
                if (out_lo + j >= non_cap) {
                    set_status(status, HL_ECAPACITY);
                    break;
                }
                const int32_t idx = indices[src_lo + j];
                non_ids[out_lo + j] = (idx < 0 || idx >= rows) ? (NonId)-1 : (NonId)(base + idx);
            }
        }
    }
    // the dense features follow their inputs: dense_out[i, :] = dense[perm[i], :] (the same threads, afterwards; a
    // launch of its own would cost more than the copy)
    if (dense != nullptr) {
        const int64_t total = (int64_t)B * n_dense;
        for (int64_t e = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; e < total;
             e += (int64_t)gridDim.x * blockDim.x) {
            const int i = (int)(e / n_dense), c = (int)(e - (int64_t)i * n_dense);
            dense_out[e] = dense[(int64_t)perm[i] * n_dense + c];
        }
    }
}

}  // namespace
}  // namespace hl

using namespace hl;

namespace hl {
namespace {

// The launches of a fragment call, for either lookup structure.  scratch: flags [max_batch], scan [n_bags + 2],
// tiles [scan_tile_words(n_bags)].
template <class Probe, typename NonId>
int32_t fragment_launch(const hl_batch* b, int T, int S, int sms, const int64_t* table_base, Probe probe,
                        uint8_t* flags, int32_t* scan, int32_t* tiles, int64_t max_bags, int32_t* status, WaitCfg waits,
                        const float* d_dense, int32_t n_dense, int32_t* d_perm, int32_t* d_counts, hl_ubatch* pop,
                        int32_t* non_offsets, NonId* non_ids, int64_t non_cap, float* d_dense_out, cudaStream_t stream) {
    const int B = b->batch;
    const int64_t n_bags = (int64_t)T * B * S;
    const bool short_bags = b->nnz <= 4 * (int64_t)T * B;   // on average at most 4 lookups per input and table
    const int cap = 4 * sms;               // CTAs of every kernel here: they stride over their work
    const int flag_grid = grid_for(B, kFlagThreads / 32, cap);
    // the tally of finished CTAs of the flags kernel: the word behind the scan's tile words (never touched by the
    // scan, zero between calls: cleared when the context is created and by the CTA that counts to the end)
    unsigned int* finished = reinterpret_cast<unsigned int*>(tiles + scan_tile_words(max_bags) - 2);
    if (short_bags)
        k_frag_flags<true, Probe><<<flag_grid, kFlagThreads, 0, stream>>>(b->indices, b->offsets, B, T, S, table_base, probe,
                                                                      flags, status, d_perm, d_counts, finished);
    else
        k_frag_flags<false, Probe><<<flag_grid, kFlagThreads, 0, stream>>>(b->indices, b->offsets, B, T, S, table_base,
                                                                       probe, flags, status, d_perm, d_counts,
                                                                       finished);
    k_frag_sizes<<<grid_for(n_bags, kThreads, cap), kThreads, 0, stream>>>(b->offsets, B, T, S, d_perm, d_counts, scan);
    note_launches(2);   // flags (with the partition), sizes
    HL_LAUNCH_CHECK();
    int32_t st = exclusive_scan_i32(scan, scan, nullptr, n_bags, tiles, status, stream, waits);
    if (st != HL_OK) return st;
    if (b->nnz <= 4 * n_bags)
        k_frag_emit<1, Probe, NonId><<<grid_for(n_bags, kThreads, cap), kThreads, 0, stream>>>(
            b->indices, b->offsets, B, T, S, d_perm, d_counts, scan, table_base, probe, pop->offsets, pop->ids,
            pop->cap_ids, non_offsets, non_ids, non_cap, status, d_dense, n_dense, d_dense_out);
    else
        k_frag_emit<32, Probe, NonId><<<grid_for(n_bags, kThreads / 32, 2 * cap), kThreads, 0, stream>>>(
            b->indices, b->offsets, B, T, S, d_perm, d_counts, scan, table_base, probe, pop->offsets, pop->ids,
            pop->cap_ids, non_offsets, non_ids, non_cap, status, d_dense, n_dense, d_dense_out);
    note_launches(1);   // emit (with the dense permutation)
    HL_LAUNCH_CHECK();
    return HL_OK;
}

}  // namespace
}  // namespace hl

extern "C" int32_t hl_fragment(hl_ctx* ctx, const hl_batch* b, const float* d_dense, int32_t n_dense,
                               int32_t* d_perm, int32_t* d_counts, hl_ubatch* pop, hl_ubatch* non,
                               float* d_dense_out, void* stream_) {
    if (!ctx || !b || !d_perm || !d_counts || !pop || !non) return HL_EINVAL;
    if (b->batch < 1 || b->batch > ctx->max_batch || b->nnz < 0 || b->nnz > ctx->max_nnz || !b->offsets ||
        (b->nnz > 0 && !b->indices))
        return HL_EINVAL;
    if (!pop->offsets || !non->offsets || (b->nnz > 0 && (!pop->ids || !non->ids))) return HL_EINVAL;
    if ((d_dense == nullptr) != (d_dense_out == nullptr) || (d_dense && n_dense < 1)) return HL_EINVAL;
    Regions& r = ctx->r;
    return fragment_launch<BitmapProbe, int32_t>(b, ctx->T, ctx->S, ctx_sms(ctx), r.table_base, BitmapProbe{r.remap},
                                                 r.frag_flags, r.frag_scan, r.frag_tiles, ctx->max_bags, r.status, wait_cfg(ctx),
                                                 d_dense, n_dense, d_perm, d_counts, pop, non->offsets, non->ids,
                                                 non->cap_ids, d_dense_out, static_cast<cudaStream_t>(stream_));
}

extern "C" int32_t hl_wide_fragment(hl_wide* w, const hl_batch* b, int32_t* d_perm, int32_t* d_counts, hl_ubatch* pop,
                                    int32_t* d_non_offsets, int64_t* d_non_rows, int64_t non_cap, void* stream_) {
    if (!w || !b || !d_perm || !d_counts || !pop || !d_non_offsets) return HL_EINVAL;
    if (b->batch < 1 || b->batch > w->max_batch || b->nnz < 0 || b->nnz > w->max_nnz || !b->offsets ||
        (b->nnz > 0 && !b->indices))
        return HL_EINVAL;
    if (!pop->offsets || (b->nnz > 0 && (!pop->ids || !d_non_rows))) return HL_EINVAL;
    const HashProbe probe{w->r_keys, w->r_vals, (uint64_t)(w->remap_slots - 1)};
    return fragment_launch<HashProbe, long long>(b, w->T, w->S, w->sms, w->table_base, probe, w->frag_flags,
                                                 w->frag_scan, w->frag_tiles, w->max_bags, w->status, WaitCfg(), nullptr, 0, d_perm,
                                                 d_counts, pop, d_non_offsets, reinterpret_cast<long long*>(d_non_rows),
                                                 non_cap, nullptr, static_cast<cudaStream_t>(stream_));
}
