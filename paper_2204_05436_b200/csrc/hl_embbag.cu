// Embedding bag over the HBM cache: sum-pooling forward, and scatter-add + SGD backward with one update per
// distinct row.  Rows are fp32 [*, D]; a group of G lanes owns one row at a time, each lane NV float4 columns,
// so that a row is read with 128-bit loads that coalesce into whole sectors.
#include <mutex>

#include "hl_common.cuh"

namespace hl {
namespace {

constexpr int kThreads = 256;

__device__ __forceinline__ float4 f4_zero() { return make_float4(0.f, 0.f, 0.f, 0.f); }

// row[0..3] += v, done by the L2 (no value comes back, so nothing waits for the row)
__device__ __forceinline__ void red_add_f4(float4* p, float4 v) {
    asm volatile("red.global.add.v4.f32 [%0], {%1, %2, %3, %4};" ::"l"(p), "f"(v.x), "f"(v.y), "f"(v.z), "f"(v.w)
                 : "memory");
}

template <int N>
__device__ __forceinline__ int32_t pick(const int32_t (&a)[N], int i) {      // a[i] without indexing registers
    int32_t r = a[0];
#pragma unroll
    for (int k = 1; k < N; ++k) r = i == k ? a[k] : r;
    return r;
}

__device__ __forceinline__ int clamp_samples(const int32_t* d_n_samples, int max_batch) {
    int n = *d_n_samples;
    if (n < 0) n = 0;
    return n < max_batch ? n : max_batch;
}

// ---- forward ------------------------------------------------------------------------------------------------
// A bag of several lookups, finished by one group of G lanes: rows are added in lookup order in fp64, four loads
// in flight, and the sum is rounded once (so cancellation between the rows of a bag costs no accuracy).
template <int G, int NV>
__device__ __forceinline__ void pool_long_bag(const float4* __restrict__ rows, const int32_t* __restrict__ ids,
                                           int32_t lo, int32_t len, int sub, int D4, int64_t n_slots,
                                           float4* __restrict__ dst, int32_t* status) {
    double acc[NV][4];
#pragma unroll
    for (int v = 0; v < NV; ++v) acc[v][0] = acc[v][1] = acc[v][2] = acc[v][3] = 0.0;
    for (int32_t p = 0; p < len; p += 4) {
        int32_t id[4];
#pragma unroll
        for (int k = 0; k < 4; ++k) id[k] = p + k < len ? __ldg(&ids[lo + p + k]) : -1;
        float4 r[4][NV];
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            const bool ok = id[k] >= 0 && id[k] < n_slots;
            if (id[k] >= n_slots) set_status(status, HL_EBOUNDS);
#pragma unroll
            for (int v = 0; v < NV; ++v) {
                const int c = sub + v * G;
                r[k][v] = (ok && c < D4) ? __ldg(&rows[(int64_t)id[k] * D4 + c]) : f4_zero();
            }
        }
#pragma unroll
        for (int k = 0; k < 4; ++k)
#pragma unroll
            for (int v = 0; v < NV; ++v) {
                acc[v][0] += (double)r[k][v].x;
                acc[v][1] += (double)r[k][v].y;
                acc[v][2] += (double)r[k][v].z;
                acc[v][3] += (double)r[k][v].w;
            }
    }
#pragma unroll
    for (int v = 0; v < NV; ++v) {
        const int c = sub + v * G;
        if (c < D4)
            __stcs(&dst[c], make_float4((float)acc[v][0], (float)acc[v][1], (float)acc[v][2], (float)acc[v][3]));
    }
}

// A group of G lanes takes UB consecutive bags per trip.  Bags of at most one lookup (the one-hot case) are plain
// row copies: the UB rows are loaded at once (UB independent 128-bit loads per lane), and the offsets and ids of
// the NEXT trip are requested before those rows are consumed, so that the offsets -> id -> row chain of one trip
// hides behind the rows of another.  Longer bags go through pool_long_bag one after the other.
template <int G, int NV, int UB>
__global__ void __launch_bounds__(kThreads, NV == 1 ? 4 : 1) k_embbag_fwd(const float* __restrict__ cache,
                                                         const int32_t* __restrict__ ids,
                                                         const int32_t* __restrict__ offsets,
                                                         const int32_t* __restrict__ d_n_samples, int max_batch,
                                                         int bags_per_sample_all /* T*S */, int D4, int64_t n_slots,
                                                         float* __restrict__ out, int32_t* status) {
    const int64_t n_bags = (int64_t)clamp_samples(d_n_samples, max_batch) * bags_per_sample_all;
    const int sub = threadIdx.x % G;
    const float4* __restrict__ rows = reinterpret_cast<const float4*>(cache);
    float4* __restrict__ out4 = reinterpret_cast<float4*>(out);

    // lo/len of the UB bags of a trip, and the id of every bag that has exactly one lookup (-1 otherwise)
    auto load_index = [&](int64_t bag0, int32_t (&lo)[UB], int32_t (&len)[UB], int32_t (&id1)[UB]) {
#pragma unroll
        for (int u = 0; u < UB; ++u) {
            const int64_t bag = bag0 + u;
            const bool valid = bag < n_bags;
            lo[u] = valid ? __ldg(&offsets[bag]) : 0;
            len[u] = valid ? __ldg(&offsets[bag + 1]) - lo[u] : -1;
        }
#pragma unroll
        for (int u = 0; u < UB; ++u) id1[u] = len[u] == 1 ? __ldg(&ids[lo[u]]) : -1;
    };

    // This CTA's share: the bags are dealt out in trips of (groups per CTA) x UB consecutive bags, every CTA gets a
    // contiguous run of trips, and the counts differ by at most one trip -- the grid is a fixed number of CTAs per
    // multiprocessor, whatever the number of bags.
    constexpr int kGroups = kThreads / G;
    int32_t lo[UB], len[UB], id1[UB];
    const int64_t trip_bags = (int64_t)kGroups * UB;
    const int64_t trips_all = (n_bags + trip_bags - 1) / trip_bags;
    const int64_t q = trips_all / gridDim.x, rem = trips_all % gridDim.x;
    const int64_t my_first = (int64_t)blockIdx.x * q + min((int64_t)blockIdx.x, rem);
    const int64_t my_trips = q + ((int64_t)blockIdx.x < rem ? 1 : 0);
    const int64_t tile0 = my_first * trip_bags;
    const int64_t tile_end = min(n_bags, tile0 + my_trips * trip_bags);
    int64_t bag0 = tile0 + (int64_t)(threadIdx.x / G) * UB;
    if (bag0 < tile_end) load_index(bag0, lo, len, id1);
    for (; bag0 < tile_end; bag0 += kGroups * UB) {
        float4 row[UB][NV];
#pragma unroll
        for (int u = 0; u < UB; ++u) {
            const bool ok = id1[u] >= 0 && id1[u] < n_slots;
            if (id1[u] >= n_slots) set_status(status, HL_EBOUNDS);
#pragma unroll
            for (int v = 0; v < NV; ++v) {
                const int c = sub + v * G;
                row[u][v] = (ok && c < D4) ? __ldg(&rows[(int64_t)id1[u] * D4 + c]) : f4_zero();
            }
        }
        int32_t cur_len[UB];
#pragma unroll
        for (int u = 0; u < UB; ++u) cur_len[u] = len[u];
        const int64_t next0 = bag0 + kGroups * UB;
        if (next0 < tile_end) load_index(next0, lo, len, id1);   // in flight while this trip's rows arrive
        unsigned long_bags = 0;   // bit u: bag u of this trip has more than one lookup
#pragma unroll
        for (int u = 0; u < UB; ++u) {
            if (cur_len[u] < 0) continue;   // past the last bag
            if (cur_len[u] > 1) {
                long_bags |= 1u << u;
                continue;
            }
            float4* dst = out4 + (bag0 + u) * D4;
#pragma unroll
            for (int v = 0; v < NV; ++v) {
                const int c = sub + v * G;
                if (c < D4) __stcs(&dst[c], row[u][v]);
            }
        }
        while (long_bags) {   // one copy of the pooling loop, whichever bag of the trip it serves
            const int u = __ffs(long_bags) - 1;
            long_bags &= long_bags - 1;
            const int64_t bag = bag0 + u;
            const int32_t b_lo = __ldg(&offsets[bag]), b_len = __ldg(&offsets[bag + 1]) - b_lo;
            pool_long_bag<G, NV>(rows, ids, b_lo, b_len, sub, D4, n_slots, out4 + bag * D4, status);
        }
    }
}

// ---- backward -----------------------------------------------------------------------------------------------
// (slot, bag) pair per lookup; a negative id becomes the sentinel n_slots, which sorts last and is ignored.
template <int GROUP>
__global__ void __launch_bounds__(kThreads) k_bwd_pairs(const int32_t* __restrict__ ids,
                                                        const int32_t* __restrict__ offsets,
                                                        const int32_t* __restrict__ d_n_samples, int max_batch,
                                                        int bags_per_sample_all, int64_t n_slots, int64_t max_nnz,
                                                        int32_t* __restrict__ keys, int32_t* __restrict__ vals,
                                                        int32_t* __restrict__ d_n_lookups,
                                                        const int32_t* __restrict__ d_pos0, int32_t key_bias,
                                                        int32_t sentinel, int32_t* __restrict__ d_total,
                                                        int32_t* status,
                                                        const int32_t* __restrict__ d_bag_bias_samples = nullptr) {
    // pairs go to positions pos0 + j (pos0 = *d_pos0 or 0) with key = slot + key_bias and value = bag (+ the bags of
    // *d_bag_bias_samples inputs, if given); *d_n_lookups = this micro-batch's lookups, *d_total (if given) = pos0 +
    // that
    const int64_t pos0 = d_pos0 ? d_pos0[0] : 0;
    const int64_t bag_bias =
        d_bag_bias_samples ? (int64_t)clamp_samples(d_bag_bias_samples, max_batch) * bags_per_sample_all : 0;
    const int64_t n_bags = (int64_t)clamp_samples(d_n_samples, max_batch) * bags_per_sample_all;
    const int sub = threadIdx.x % GROUP;
    const int64_t group = ((int64_t)blockIdx.x * kThreads + threadIdx.x) / GROUP;
    const int64_t n_groups = (int64_t)gridDim.x * kThreads / GROUP;
    if (group == 0 && sub == 0) {
        int32_t L = offsets[n_bags];
        if (pos0 + L > max_nnz) {
            set_status(status, HL_ECAPACITY);
            L = (int32_t)(max_nnz - pos0);
        }
        d_n_lookups[0] = L;
        if (d_total) d_total[0] = (int32_t)(pos0 + L);
    }
    for (int64_t bag = group; bag < n_bags; bag += n_groups) {
        const int32_t lo = offsets[bag], hi = offsets[bag + 1];
        for (int32_t j = lo + sub; j < hi; j += GROUP) {
            if (pos0 + j >= max_nnz) break;
            const int32_t id = ids[j];
            if (id >= n_slots) set_status(status, HL_EBOUNDS);
            keys[pos0 + j] = (id < 0 || id >= n_slots) ? sentinel : id + key_bias;
            vals[pos0 + j] = (int32_t)(bag + bag_bias);
        }
    }
}

// The sorted lookups are cut into chunks of kBwdChunk.  One group per chunk sums, in order, the gradient rows of
// each run of equal slots inside its chunk.  A run that lies wholly inside the chunk is finished here (one
// reduction into its row).  A run that crosses a chunk border leaves a partial sum: part[chunk][0] for the
// piece that continues a run from the previous chunk, part[chunk][1] for the piece that starts a run continuing
// into the next chunk.  k_bwd_spans adds those up.
//
// The group reads its chunk's 32 (slot, bag) pairs with one coalesced load per lane.  Where runs begin and end is
// then settled once for the whole chunk: every lane compares its pairs' slots with their neighbours' (shuffles, the
// slots just outside the chunk for the ends) and two ballots per 32 pairs give a mask of run heads and a mask of
// run tails.  The loop over the lookups is driven by those two masks alone, and a lookup costs two shuffles, one
// address, one 128-bit load per column and the additions; everything that checks a pair (position inside the call,
// bag inside the gradient array) is done by the lane that loaded the pair, once.  Gradient rows are loaded U at a
// time.  The instruction count matters: this kernel issues about as many cycles as it waits for memory.
//
// A run that starts in one chunk and ends in the next (most runs that cross a border do) is finished by the group of
// the chunk it starts in, which reads on into the next chunk; the group of that next chunk leaves the run's lookups
// alone.  Both decide from the sorted slots alone and by the same test -- the run's head lies in the first of the two
// chunks, and the chunk after the second does not begin with the run's slot -- so exactly one of them sums each
// lookup.  Only runs over three or more chunks go through partial sums and k_bwd_spans.
static_assert(kBwdChunk == 32, "the head and tail masks of a chunk are 32-bit words");

template <int G, int NV>
__global__ void __launch_bounds__(kThreads, NV == 1 ? 3 : 1) k_bwd_chunks(float* __restrict__ cache,
                                                         const int32_t* __restrict__ keys,
                                                         const int32_t* __restrict__ vals,
                                                         const int32_t* __restrict__ d_n_lookups,
                                                         const float* __restrict__ grad_out, int D4, int64_t n_slots,
                                                         float lr, float* __restrict__ part,
                                                         const int32_t* __restrict__ d_first, int32_t key_bias,
                                                         int32_t* __restrict__ span_count,
                                                         int32_t* __restrict__ span_list, int64_t n_grad_rows,
                                                         int64_t max_entries, int32_t* status) {
    // the lookups of this call are positions [first, first + *d_n_lookups) of the sorted arrays; their keys are
    // slot + key_bias.  A chunk in which a run starts that goes on into the next chunk is appended to span_list
    // (in any order): k_bwd_spans finishes those runs.
    constexpr int KPL = kBwdChunk / G;                       // pairs held per lane
    constexpr int U = NV >= 4 ? 2 : (NV >= 2 ? 4 : (G >= 8 ? 8 : 4));       // lookups in flight per lane
    static_assert(G % U == 0, "batch must divide the group");
    const int64_t first = d_first ? d_first[0] : 0;
    const int64_t n = first + d_n_lookups[0];
    const int lane = threadIdx.x & 31;
    const int sub = lane % G;
    const unsigned gshift = G == 32 ? 0u : (unsigned)(lane / G * G);
    constexpr unsigned gbits = G == 32 ? 0xffffffffu : ((1u << G) - 1u);
    const unsigned gmask = gbits << gshift;
    const int64_t group = ((int64_t)blockIdx.x * kThreads + threadIdx.x) / G;
    const int64_t n_groups = (int64_t)gridDim.x * kThreads / G;
    float4* cache4 = reinterpret_cast<float4*>(cache);
    float4* __restrict__ part4 = reinterpret_cast<float4*>(part);
    // slots and bags are 32-bit numbers, so one unsigned comparison tells whether one lies inside its array
    const uint32_t n_rows_u = (uint32_t)(n_slots < 0x7fffffff ? n_slots : 0x7fffffff);
    const uint32_t n_grad_u = (uint32_t)(n_grad_rows < 0x7fffffff ? n_grad_rows : 0x7fffffff);
    // this lane's columns; a lane beyond the row's width reads column 0 and writes nothing
    bool on[NV];
    const float4* gcol[NV];
#pragma unroll
    for (int v = 0; v < NV; ++v) {
        const int c = sub + v * G;
        on[v] = c < D4;
        gcol[v] = reinterpret_cast<const float4*>(grad_out) + (on[v] ? c : 0);
    }

    for (int64_t chunk = group; first + chunk * kBwdChunk < n; chunk += n_groups) {
        const int64_t start = first + chunk * kBwdChunk;
        const int64_t end = min(start + (int64_t)kBwdChunk, n);
        int32_t kk[KPL], vv[KPL];
#pragma unroll
        for (int i = 0; i < KPL; ++i) {
            const int64_t p = start + i * G + sub;
            const bool in = p < end;
            kk[i] = in ? keys[p] : -1;                       // -1: past the end; no slot has this key
            const int32_t bag = in ? vals[p] : 0;
            // (a bag id outside the gradient array can only be what a given-up chain poll of the sort left behind;
            // such a call has its error status set, and reads bag 0 instead)
            vv[i] = (uint32_t)bag < n_grad_u ? bag : 0;
        }
        const int32_t prev_key = start > first ? keys[start - 1] : -3;   // -3: equal to no key
        const int32_t next_key = end < n ? keys[end] : -2;
        // the slot before the previous chunk, and the first slot of the chunk after the next one
        const int32_t prev2_key = start - kBwdChunk > first ? keys[start - kBwdChunk - 1] : -3;
        const int32_t next2_key = start + 2 * kBwdChunk < n ? keys[start + 2 * kBwdChunk] : -2;

        // bit q of `heads`: lookup q of the chunk begins a run; of `tails`: it ends one
        uint32_t heads = 0, tails = 0;
#pragma unroll
        for (int i = 0; i < KPL; ++i) {
            const int32_t up = __shfl_up_sync(gmask, kk[i], 1, G);
            const int32_t dn = __shfl_down_sync(gmask, kk[i], 1, G);
            const int32_t before = i > 0 ? __shfl_sync(gmask, kk[i > 0 ? i - 1 : 0], G - 1, G) : prev_key;
            const int32_t after = i + 1 < KPL ? __shfl_sync(gmask, kk[i + 1 < KPL ? i + 1 : i], 0, G) : next_key;
            const int32_t pred = sub > 0 ? up : before;
            const int32_t succ = sub < G - 1 ? dn : after;
            const uint32_t hb = (__ballot_sync(gmask, kk[i] != pred) >> gshift) & gbits;
            const uint32_t tb = (__ballot_sync(gmask, kk[i] != succ) >> gshift) & gbits;
            heads |= hb << (i * G);
            tails |= tb << (i * G);
        }

        const bool ends_open = !((tails >> (kBwdChunk - 1)) & 1u);   // the last run goes on in the next chunk
        // A run that comes in from the previous chunk, began there and ends here was finished by that chunk's group:
        // its lookups (up to its tail, the lowest tail bit) are not summed here -- their loads are pointed at the bag
        // of the chunk's last lookup, which is loaded anyway, and the tail bit is cleared so that nothing is applied.
        {
            const int32_t key0 = __shfl_sync(gmask, kk[0], 0, G);
            if (chunk >= 1 && !(heads & 1u) && tails != 0u && prev2_key != key0) {
                const int t = __ffs((int)tails) - 1;
                tails &= tails - 1u;
                const int32_t last_bag = __shfl_sync(gmask, vv[KPL - 1], G - 1, G);
#pragma unroll
                for (int i = 0; i < KPL; ++i)
                    if (i * G + sub <= t) vv[i] = last_bag;
            }
        }

        // the run being summed continues one from the previous chunk until the first head
        bool left_open = true;
        // a segment's sum is kept in fp64: a popular row can collect tens of thousands of gradient rows, and the
        // rounding of many fp32 partial sums would show in the updated row
        double acc[NV][4];
#pragma unroll
        for (int v = 0; v < NV; ++v) acc[v][0] = acc[v][1] = acc[v][2] = acc[v][3] = 0.0;

        // the run whose last lookup in this chunk has key `key` is complete in acc
        auto emit = [&](int32_t key, bool right_open) {
            const uint32_t row = (uint32_t)(key - key_bias);
            if (row >= n_rows_u) return;                     // a skipped lookup's sentinel, or past the end
            if (!left_open && !right_open) {
#pragma unroll
                for (int v = 0; v < NV; ++v)
                    if (on[v])
                        red_add_f4(&cache4[(int64_t)row * D4 + sub + v * G],
                                   make_float4(-(lr * (float)acc[v][0]), -(lr * (float)acc[v][1]),
                                               -(lr * (float)acc[v][2]), -(lr * (float)acc[v][3])));
            } else {
                const int64_t slot = chunk * 2 + (left_open ? 0 : 1);
#pragma unroll
                for (int v = 0; v < NV; ++v)
                    if (on[v])
                        part4[slot * D4 + sub + v * G] =
                            make_float4((float)acc[v][0], (float)acc[v][1], (float)acc[v][2], (float)acc[v][3]);
                if (right_open && !left_open) {
                    // a run starts here and goes on: list it, with its last chunk if that is among the next G (chunk
                    // c > chunk holds a piece of the run iff its first slot is the run's; sorted keys: those chunks
                    // form a prefix).  Nearly every run ends there, and k_bwd_spans then has nothing to search.
                    const int64_t n_chunks = (n - first + kBwdChunk - 1) / kBwdChunk;
                    const int64_t cc = chunk + 1 + sub;
                    const bool goes_on = cc < n_chunks && keys[first + cc * kBwdChunk] == key;
                    const uint32_t m = (__ballot_sync(gmask, goes_on) >> gshift) & gbits;
                    const int cnt = __ffs((int)~m) - 1;      // m == gbits (all G go on): -1 for G == 32, else G
                    if (sub == 0) {
                        const int32_t pos = atomicAdd(span_count, 1);
                        // (one entry per chunk at most, and the count is zero when a call starts: the list cannot
                        // overflow unless an earlier call was cut short between its two kernels)
                        if (pos >= 0 && pos < max_entries)
                            reinterpret_cast<int4*>(span_list)[pos] =
                                make_int4((int32_t)chunk, key, (cnt >= 1 && cnt < G) ? (int32_t)(chunk + cnt) : -1, 0);
                        else
                            set_status(status, HL_ECAPACITY);
                    }
                }
            }
        };

#pragma unroll
        for (int i = 0; i < KPL; ++i) {
            // (kept rolled: with all 32 lookups unrolled the kernel is tens of KB of straight-line code that every
            // warp runs through about once, and it waits for instructions)
#pragma unroll 1
            for (int j = 0; j < G; j += U) {
                int32_t k[U];
                float4 g[U][NV];
#pragma unroll
                for (int u = 0; u < U; ++u) {
                    k[u] = __shfl_sync(gmask, kk[i], j + u, G);
                    const int32_t bag = __shfl_sync(gmask, vv[i], j + u, G);
#pragma unroll
                    for (int v = 0; v < NV; ++v) g[u][v] = __ldg(gcol[v] + (int64_t)bag * D4);
                }
#pragma unroll
                for (int u = 0; u < U; ++u) {
                    const int q = i * G + j + u;
                    if ((heads >> q) & 1u) {
                        left_open = false;
#pragma unroll
                        for (int v = 0; v < NV; ++v) acc[v][0] = acc[v][1] = acc[v][2] = acc[v][3] = 0.0;
                    }
#pragma unroll
                    for (int v = 0; v < NV; ++v) {
                        acc[v][0] += (double)g[u][v].x;
                        acc[v][1] += (double)g[u][v].y;
                        acc[v][2] += (double)g[u][v].z;
                        acc[v][3] += (double)g[u][v].w;
                    }
                    if ((tails >> q) & 1u) emit(k[u], false);
                }
            }
        }
        // the chunk's last lookup does not end its run: the run goes on in the next chunk (only a full chunk has a
        // next one)
        if (ends_open) {
            const int32_t key = __shfl_sync(gmask, kk[KPL - 1], G - 1, G);
            if (!left_open && next2_key != key && (uint32_t)(key - key_bias) < n_rows_u) {
                // it began in this chunk and ends in the next: its lookups there are summed here as well (they are a
                // prefix of that chunk: m of them), and the row gets its one update
                const int64_t start2 = start + kBwdChunk;
                const int64_t end2 = min(start2 + (int64_t)kBwdChunk, n);
                int32_t vv2[KPL];
                uint32_t same = 0;
#pragma unroll
                for (int i = 0; i < KPL; ++i) {
                    const int64_t p = start2 + i * G + sub;
                    const bool in = p < end2;
                    const int32_t k2 = in ? keys[p] : -1;
                    const int32_t bag = in ? vals[p] : 0;
                    vv2[i] = (uint32_t)bag < n_grad_u ? bag : 0;
                    same |= ((__ballot_sync(gmask, k2 == key) >> gshift) & gbits) << (i * G);
                }
                const int m = same == 0xffffffffu ? kBwdChunk : __ffs((int)~same) - 1;
#pragma unroll 1
                for (int q0 = 0; q0 < m; q0 += U) {
                    float4 g[U][NV];
#pragma unroll
                    for (int u = 0; u < U; ++u) {
                        const int q = q0 + u < m ? q0 + u : m - 1;       // (past the run's end: a row already asked for)
                        const int32_t bag = __shfl_sync(gmask, pick(vv2, q / G), q % G, G);
#pragma unroll
                        for (int v = 0; v < NV; ++v) g[u][v] = __ldg(gcol[v] + (int64_t)bag * D4);
                    }
#pragma unroll
                    for (int u = 0; u < U; ++u) {
                        if (q0 + u >= m) continue;
#pragma unroll
                        for (int v = 0; v < NV; ++v) {
                            acc[v][0] += (double)g[u][v].x;
                            acc[v][1] += (double)g[u][v].y;
                            acc[v][2] += (double)g[u][v].z;
                            acc[v][3] += (double)g[u][v].w;
                        }
                    }
                }
                emit(key, false);
            } else {
                emit(key, true);
            }
        }
    }
}

// One WARP per chunk; it acts only if a run STARTS in its chunk and continues into the next one.  The lanes look
// at the first slot of the next 32 chunks at once to find where the run ends (and, if it goes on, close in on the end
// with a 32-way search over the rest of the list).  A run of up to kLongRun chunks is summed by its warp: the 32/G
// groups add the run's continuation pieces in an interleaved, fixed order in fp64 (runs of many thousands of lookups
// occur), the group sums are combined by shuffles in a fixed order, and group 0 applies the single SGD update of the
// row.  Longer runs (a popular row can own hundreds of chunks) are queued in shared memory and then summed by the
// whole CTA, every group taking every (8 * 32/G)-th piece, the group sums combined in a fixed order by one group.
constexpr int kLongRun = 32;

template <int G, int NV>
__global__ void __launch_bounds__(kThreads) k_bwd_spans(float* __restrict__ cache, const int32_t* __restrict__ keys,
                                                        const int32_t* __restrict__ d_n_lookups, int D4,
                                                        int64_t n_slots, float lr, const float* __restrict__ part,
                                                        const int32_t* __restrict__ d_first, int32_t key_bias,
                                                        int32_t* span_count,
                                                        const int32_t* __restrict__ span_list, int64_t max_entries) {
    constexpr int GW = 32 / G;   // groups per warp
    constexpr int kWarps = kThreads / 32;
    constexpr int U = NV >= 4 ? 2 : (NV >= 2 ? 4 : 8);   // partial sums in flight per lane
    constexpr int UC = 8;                // the same in the CTA-wide sum
    constexpr bool kCtaPath = NV == 1;   // the CTA-wide sum keeps one float4 column per lane
    __shared__ int64_t q_chunk[kWarps], q_last[kWarps], q_row[kWarps];
    __shared__ double s_sum[kCtaPath ? kThreads : 1][4];
    const int64_t first = d_first ? d_first[0] : 0;
    const int64_t n = first + d_n_lookups[0];
    const int lane = threadIdx.x & 31, wib = threadIdx.x >> 5;
    const int sub = lane % G, gi = lane / G;
    const float4* __restrict__ part4 = reinterpret_cast<const float4*>(part);
    float4* cache4 = reinterpret_cast<float4*>(cache);
    const int64_t n_chunks = (n - first + kBwdChunk - 1) / kBwdChunk;

    int64_t n_owned = span_count[0];     // chunks in which a run starts that goes on into the next chunk
    n_owned = n_owned < 0 ? 0 : (n_owned < n_chunks ? n_owned : n_chunks);
    n_owned = n_owned < max_entries ? n_owned : max_entries;

    // every warp of the CTA makes the same number of trips (there are block barriers inside)
    for (int64_t base = (int64_t)blockIdx.x * kWarps; base < n_owned; base += (int64_t)gridDim.x * kWarps) {
        if (kCtaPath && lane == 0) q_chunk[wib] = -1;
        bool mine = false;
        int32_t key = 0;
        int64_t chunk = 0, row = 0, last_chunk = 0;
        int64_t known_last = -1;
        if (base + wib < n_owned) {
            // (chunk, slot key of the run, its last chunk if the sum kernel has found it)
            const int4 e = reinterpret_cast<const int4*>(span_list)[base + wib];
            chunk = e.x;
            key = e.y;
            row = (int64_t)key - key_bias;
            mine = chunk >= 0 && chunk + 1 < n_chunks && row >= 0 && row < n_slots;
            if (e.z > e.x && e.z < n_chunks) known_last = e.z;
        }
        // the run's first piece is asked for now; it is needed after the search
        float4 piece0[NV];
#pragma unroll
        for (int v = 0; v < NV; ++v) {
            const int c = sub + v * G;
            const bool ld = mine && gi == 0 && c < D4;
            piece0[v] = ld ? part4[(chunk * 2 + 1) * D4 + c] : f4_zero();
        }
        if (mine) {
            // last chunk that holds a piece of the run: chunk c > chunk holds one iff its first slot is the run's
            int64_t lo = chunk + 1, hi = n_chunks;      // chunk lo holds a piece, chunk hi (if any) does not
            if (known_last >= 0) {
                lo = known_last;
                hi = known_last + 1;
            } else {
                const int64_t cc = lo + 1 + lane;       // the 32 chunks after lo
                const bool t = cc < hi && keys[first + cc * kBwdChunk] == key;
                const unsigned m = __ballot_sync(0xffffffffu, t);
                const int cnt = __popc(m);              // sorted keys: the lanes that see the run form a prefix
                lo += cnt;
                if (cnt < 32) hi = min(hi, lo + 1);
            }
            while (hi - lo > 1) {
                const int64_t step = (hi - lo + 31) / 32;
                const int64_t cc = lo + (lane + 1) * step;
                const bool t = cc < hi && keys[first + cc * kBwdChunk] == key;
                const int cnt = __popc(__ballot_sync(0xffffffffu, t));
                const int64_t new_hi = min(hi, lo + (cnt + 1) * step);
                lo += cnt * step;
                hi = new_hi;
            }
            last_chunk = lo;
            if (kCtaPath && last_chunk - chunk > kLongRun) {
                if (lane == 0) {
                    q_chunk[wib] = chunk;
                    q_last[wib] = last_chunk;
                    q_row[wib] = row;
                }
                mine = false;        // summed by the whole CTA below
            }
        }
        if (mine) {
            double dacc[NV][4];
#pragma unroll
            for (int v = 0; v < NV; ++v) {
                dacc[v][0] = piece0[v].x;
                dacc[v][1] = piece0[v].y;
                dacc[v][2] = piece0[v].z;
                dacc[v][3] = piece0[v].w;
            }
            for (int64_t c2 = chunk + 1 + gi; c2 <= last_chunk; c2 += (int64_t)GW * U) {
                float4 t[U][NV];
#pragma unroll
                for (int u = 0; u < U; ++u)
#pragma unroll
                    for (int v = 0; v < NV; ++v) {
                        const int c = sub + v * G;
                        const int64_t cc = c2 + (int64_t)u * GW;
                        t[u][v] = (cc <= last_chunk && c < D4) ? part4[(cc * 2) * D4 + c] : f4_zero();
                    }
#pragma unroll
                for (int u = 0; u < U; ++u)
#pragma unroll
                    for (int v = 0; v < NV; ++v) {
                        dacc[v][0] += (double)t[u][v].x;
                        dacc[v][1] += (double)t[u][v].y;
                        dacc[v][2] += (double)t[u][v].z;
                        dacc[v][3] += (double)t[u][v].w;
                    }
            }
#pragma unroll
            for (int off = G; off < 32; off <<= 1)
#pragma unroll
                for (int v = 0; v < NV; ++v)
#pragma unroll
                    for (int e = 0; e < 4; ++e) dacc[v][e] += __shfl_xor_sync(0xffffffffu, dacc[v][e], off);
            if (gi == 0) {
#pragma unroll
                for (int v = 0; v < NV; ++v) {
                    const int c = sub + v * G;
                    if (c < D4)
                        red_add_f4(&cache4[row * D4 + c],
                                   make_float4(-(lr * (float)dacc[v][0]), -(lr * (float)dacc[v][1]),
                                               -(lr * (float)dacc[v][2]), -(lr * (float)dacc[v][3])));
                }
            }
        }
        if (kCtaPath) {
            __syncthreads();
            for (int qi = 0; qi < kWarps; ++qi) {
                const int64_t qc = q_chunk[qi];
                if (qc < 0) continue;                    // the same for all threads
                const int64_t ql = q_last[qi], qrow = q_row[qi];
                const int gg = wib * GW + gi;            // this group among the CTA's kWarps * GW groups
                double d0 = 0.0, d1 = 0.0, d2 = 0.0, d3 = 0.0;
                for (int64_t c2 = qc + 1 + gg; c2 <= ql; c2 += (int64_t)kWarps * GW * UC) {
                    float4 t[UC];
#pragma unroll
                    for (int u = 0; u < UC; ++u) {
                        const int64_t cc = c2 + (int64_t)u * kWarps * GW;
                        t[u] = (cc <= ql && sub < D4) ? part4[(cc * 2) * D4 + sub] : f4_zero();
                    }
#pragma unroll
                    for (int u = 0; u < UC; ++u) {
                        d0 += (double)t[u].x;
                        d1 += (double)t[u].y;
                        d2 += (double)t[u].z;
                        d3 += (double)t[u].w;
                    }
                }
                s_sum[threadIdx.x][0] = d0;
                s_sum[threadIdx.x][1] = d1;
                s_sum[threadIdx.x][2] = d2;
                s_sum[threadIdx.x][3] = d3;
                __syncthreads();
                if (threadIdx.x < G && sub < D4) {       // group 0 of warp 0: lane sub owns column sub
                    const float4 p = part4[(qc * 2 + 1) * D4 + sub];      // the piece in the run's first chunk
                    double a0 = p.x, a1 = p.y, a2 = p.z, a3 = p.w;
                    for (int g2 = 0; g2 < kWarps * GW; ++g2) {
                        a0 += s_sum[g2 * G + sub][0];
                        a1 += s_sum[g2 * G + sub][1];
                        a2 += s_sum[g2 * G + sub][2];
                        a3 += s_sum[g2 * G + sub][3];
                    }
                    red_add_f4(&cache4[qrow * D4 + sub], make_float4(-(lr * (float)a0), -(lr * (float)a1),
                                                                     -(lr * (float)a2), -(lr * (float)a3)));
                }
                __syncthreads();
            }
            __syncthreads();     // every warp has read the whole queue before any warp clears its entry again
        }
    }
    // The list is empty again for the next call: the last CTA to get here clears the count (word 0) and the tally of
    // finished CTAs (word 2).  Every CTA read the count when it started, and the next call's kernels start after this
    // grid has ended.
    __syncthreads();
    if (threadIdx.x == 0) {
        const int32_t finished = atomicAdd(&span_count[2], 1);
        if (finished == (int32_t)gridDim.x - 1) {
            span_count[0] = 0;
            span_count[2] = 0;
        }
    }
}

template <int G, int NV>
int32_t launch_fwd(hl_ctx* ctx, const float* cache, const hl_ubatch* ub, const int32_t* d_n, float* out,
                   cudaStream_t stream) {
    constexpr int UB = NV >= 4 ? 1 : (NV >= 2 ? 2 : 4);
    const int64_t bags_per_trip = (int64_t)(kThreads / G) * UB;
    const int grid = grid_for(ctx->max_bags, (int)bags_per_trip, fwd_ctas_per_sm(ctx) * ctx_sms(ctx));
    timer_mark(ctx, HL_TIMER_FWD, 0, stream);
    k_embbag_fwd<G, NV, UB><<<grid, kThreads, 0, stream>>>(cache, ub->ids, ub->offsets, d_n, ctx->max_batch,
                                                          ctx->T * ctx->S, ctx->D / 4,
                                                          ctx->hot_cap + ctx->staging_cap, out, ctx->r.status);
    timer_mark(ctx, HL_TIMER_FWD, 1, stream);
    note_launches(1);
    HL_LAUNCH_CHECK();
    return HL_OK;
}

template <int G, int NV>
int32_t launch_bwd(hl_ctx* ctx, float* cache, const int32_t* keys, const int32_t* vals, const int32_t* d_n_lookups,
                   const float* grad, float lr, cudaStream_t stream, const int32_t* d_first = nullptr,
                   int32_t key_bias = 0) {
    const int64_t max_chunks = div_up(ctx->max_nnz, kBwdChunk);
    // a fixed number of CTAs per multiprocessor (the groups stride over the chunks), so that kernels of other
    // streams find room beside this one
    const int grid = grid_for(max_chunks * G, kThreads, bwd_ctas_per_sm(ctx) * ctx_sms(ctx));
    const int64_t n_slots = ctx->hot_cap + ctx->staging_cap;
    timer_mark(ctx, HL_TIMER_BWD_REDUCE, 0, stream);
    // the list of runs that cross a chunk border sits behind the partial sums: [count words (8 ints)] [entries].
    // The count is zero between calls: hl_create clears it and k_bwd_spans clears it again when it is done.
    int32_t* span_count = span_count_of(ctx);
    int32_t* span_list = span_count + 8;
    k_bwd_chunks<G, NV><<<grid, kThreads, 0, stream>>>(cache, keys, vals, d_n_lookups, grad, ctx->D / 4, n_slots,
                                                      lr, ctx->r.bwd_part, d_first, key_bias, span_count, span_list,
                                                      ctx->max_bags, max_chunks, ctx->r.status);
    timer_mark(ctx, HL_TIMER_BWD_REDUCE, 1, stream);
    const int span_grid = grid_for(max_chunks * 32, kThreads, 4 * ctx_sms(ctx));   // the warps stride over the listed runs
    k_bwd_spans<G, NV><<<span_grid, kThreads, 0, stream>>>(cache, keys, d_n_lookups, ctx->D / 4, n_slots, lr,
                                                          ctx->r.bwd_part, d_first, key_bias, span_count,
                                                          (const int32_t*)span_list, max_chunks);
    note_launches(2);
    HL_LAUNCH_CHECK();
    return HL_OK;
}

int bits_for(int64_t max_value) {
    int b = 1;
    while ((int64_t(1) << b) <= max_value) ++b;
    return b;
}

}  // namespace
}  // namespace hl

using namespace hl;

#define HL_DISPATCH_ROW_SHAPE(D4, CALL)                  \
    do {                                                 \
        if ((D4) <= 4) return CALL(4, 1);                \
        if ((D4) <= 8) return CALL(8, 1);                \
        if ((D4) <= 16) return CALL(16, 1);              \
        if ((D4) <= 32) return CALL(32, 1);              \
        if ((D4) <= 64) return CALL(32, 2);              \
        if ((D4) <= 128) return CALL(32, 4);             \
        if ((D4) <= 256) return CALL(32, 8);             \
        return HL_EINVAL;                                \
    } while (0)

extern "C" int32_t hl_embbag_fwd(hl_ctx* ctx, const float* d_cache, const hl_ubatch* ub, const int32_t* d_n_samples,
                                 float* d_out, void* stream_) {
    if (!ctx || !d_cache || !ub || !ub->offsets || !d_n_samples || !d_out) return HL_EINVAL;
    if (ctx->max_nnz > 0 && !ub->ids) return HL_EINVAL;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
#define HL_FWD(G, NV) launch_fwd<G, NV>(ctx, d_cache, ub, d_n_samples, d_out, stream)
    HL_DISPATCH_ROW_SHAPE(ctx->D / 4, HL_FWD);
#undef HL_FWD
}

namespace hl {
namespace {

// (slot, bag) pairs of the micro-batch, sorted by slot (stable).  The result lands in out_keys / out_vals: either
// the caller's arrays (which then serve as one half of the sort's ping-pong buffers) or, if they are null, whichever
// scratch buffer the last pass wrote.
int32_t sort_lookups(hl_ctx* ctx, const hl_ubatch* ub, const int32_t* d_n_samples, int32_t* caller_keys,
                     int32_t* caller_vals, int32_t* d_n_lookups, int32_t** out_keys, int32_t** out_vals,
                     cudaStream_t stream) {
    Regions& r = ctx->r;
    const int64_t n_slots = ctx->hot_cap + ctx->staging_cap;
    const int key_bits = bits_for(n_slots);
    const int passes = (key_bits + 7) / 8;
    int32_t* keys[2] = {r.bwd_keys[0], r.bwd_keys[1]};
    int32_t* vals[2] = {r.bwd_vals[0], r.bwd_vals[1]};
    if (caller_keys) {   // make the buffer the last pass writes the caller's
        keys[passes & 1] = caller_keys;
        vals[passes & 1] = caller_vals;
    }
    const bool short_bags = ctx->max_nnz <= 4 * ctx->max_bags;
    if (short_bags)
        k_bwd_pairs<1><<<grid_for(ctx->max_bags, kThreads, 4 * ctx_sms(ctx)), kThreads, 0, stream>>>(
            ub->ids, ub->offsets, d_n_samples, ctx->max_batch, ctx->T * ctx->S, n_slots, ctx->max_nnz, keys[0], vals[0],
            d_n_lookups, nullptr, 0, (int32_t)n_slots, nullptr, r.status);
    else
        k_bwd_pairs<32><<<grid_for(ctx->max_bags, kThreads / 32, 8 * ctx_sms(ctx)), kThreads, 0, stream>>>(
            ub->ids, ub->offsets, d_n_samples, ctx->max_batch, ctx->T * ctx->S, n_slots, ctx->max_nnz, keys[0], vals[0],
            d_n_lookups, nullptr, 0, (int32_t)n_slots, nullptr, r.status);
    note_launches(1);
    HL_LAUNCH_CHECK();
    return radix_sort_pairs(keys, vals, d_n_lookups, ctx->max_nnz, key_bits, r.bwd_hist, r.status, out_keys, out_vals,
                            stream, wait_cfg(ctx));
}

}  // namespace
}  // namespace hl

extern "C" int32_t hl_embbag_bwd_sgd(hl_ctx* ctx, float* d_cache, const hl_ubatch* ub, const int32_t* d_n_samples,
                                     const float* d_grad_out, float lr, void* stream_) {
    if (!ctx || !d_cache || !ub || !ub->offsets || !d_n_samples || !d_grad_out) return HL_EINVAL;
    if (ctx->max_nnz == 0) return HL_OK;
    if (!ub->ids) return HL_EINVAL;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    int32_t *keys, *vals;
    int32_t st = sort_lookups(ctx, ub, d_n_samples, nullptr, nullptr, ctx->r.bwd_n, &keys, &vals, stream);
    if (st != HL_OK) return st;
#define HL_BWD(G, NV) launch_bwd<G, NV>(ctx, d_cache, keys, vals, ctx->r.bwd_n, d_grad_out, lr, stream)
    HL_DISPATCH_ROW_SHAPE(ctx->D / 4, HL_BWD);
#undef HL_BWD
}

extern "C" int32_t hl_embbag_bwd_prepare(hl_ctx* ctx, const hl_ubatch* ub, const int32_t* d_n_samples,
                                         int32_t* d_sorted_slots, int32_t* d_sorted_bags, int32_t* d_n_lookups,
                                         void* stream_) {
    if (!ctx || !ub || !ub->offsets || !d_n_samples || !d_n_lookups) return HL_EINVAL;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    if (ctx->max_nnz == 0) {
        HL_CUDA_TRY(cudaMemsetAsync(d_n_lookups, 0, sizeof(int32_t), stream));
        return HL_OK;
    }
    if (!ub->ids || !d_sorted_slots || !d_sorted_bags) return HL_EINVAL;
    int32_t *keys, *vals;
    return sort_lookups(ctx, ub, d_n_samples, d_sorted_slots, d_sorted_bags, d_n_lookups, &keys, &vals, stream);
}

static int32_t prepare_both(hl_ctx* ctx, const hl_ubatch* pop, const int32_t* d_n_pop, const hl_ubatch* non,
                            const int32_t* d_n_non, int32_t* d_sorted_slots, int32_t* d_sorted_bags,
                            int32_t* d_n_lookups, bool merge, void* stream_) {
    // merge = false: X's keys are offset by the number of slots + 1, so that the sorted list is O's pairs (skipped
    // lookups of O, key n_slots, last among them), then X's (its skipped lookups, key 2 * n_slots + 1, at the very end);
    // merge = true: one key space, and X's bags are numbered behind O's: the lookups of a row from both
    // micro-batches form one run, over one gradient array [bags of O; bags of X]
    if (!ctx || !pop || !non || !pop->offsets || !non->offsets || !d_n_pop || !d_n_non || !d_n_lookups)
        return HL_EINVAL;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    if (ctx->max_nnz == 0) {
        HL_CUDA_TRY(cudaMemsetAsync(d_n_lookups, 0, 4 * sizeof(int32_t), stream));
        return HL_OK;
    }
    if (!pop->ids || !non->ids || !d_sorted_slots || !d_sorted_bags) return HL_EINVAL;
    Regions& r = ctx->r;
    const int64_t n_slots = ctx->hot_cap + ctx->staging_cap;
    if (2 * n_slots + 2 >= (int64_t(1) << 31)) return HL_EINVAL;
    const int key_bits = bits_for(merge ? n_slots : 2 * n_slots + 1);
    const int passes = (key_bits + 7) / 8;
    int32_t* keys[2] = {r.bwd_keys[0], r.bwd_keys[1]};
    int32_t* vals[2] = {r.bwd_vals[0], r.bwd_vals[1]};
    keys[passes & 1] = d_sorted_slots;
    vals[passes & 1] = d_sorted_bags;
    const bool short_bags = ctx->max_nnz <= 4 * ctx->max_bags;
    const int per_block = short_bags ? kThreads : kThreads / 32;
    const int grid = grid_for(ctx->max_bags, per_block, (short_bags ? 4 : 8) * ctx_sms(ctx));
    const hl_ubatch* ubs[2] = {pop, non};
    const int32_t* ns[2] = {d_n_pop, d_n_non};
    for (int m = 0; m < 2; ++m) {
        const int32_t* pos0 = m == 0 ? nullptr : d_n_lookups;
        const int32_t bias = (m == 0 || merge) ? 0 : (int32_t)(n_slots + 1);
        const int32_t sentinel = bias + (int32_t)n_slots;
        const int32_t* bag_bias = (m == 1 && merge) ? d_n_pop : nullptr;
        if (short_bags)
            k_bwd_pairs<1><<<grid, kThreads, 0, stream>>>(ubs[m]->ids, ubs[m]->offsets, ns[m], ctx->max_batch,
                                                         ctx->T * ctx->S, n_slots, ctx->max_nnz, keys[0], vals[0],
                                                         d_n_lookups + m, pos0, bias, sentinel, d_n_lookups + 2,
                                                         r.status, bag_bias);
        else
            k_bwd_pairs<32><<<grid, kThreads, 0, stream>>>(ubs[m]->ids, ubs[m]->offsets, ns[m], ctx->max_batch,
                                                          ctx->T * ctx->S, n_slots, ctx->max_nnz, keys[0], vals[0],
                                                          d_n_lookups + m, pos0, bias, sentinel, d_n_lookups + 2,
                                                          r.status, bag_bias);
    }
    note_launches(2);
    HL_LAUNCH_CHECK();
    int32_t *ok, *ov;
    return radix_sort_pairs(keys, vals, d_n_lookups + 2, ctx->max_nnz, key_bits, r.bwd_hist, r.status, &ok, &ov, stream,
                            wait_cfg(ctx));
}

extern "C" int32_t hl_embbag_bwd_prepare2(hl_ctx* ctx, const hl_ubatch* pop, const int32_t* d_n_pop,
                                          const hl_ubatch* non, const int32_t* d_n_non, int32_t* d_sorted_slots,
                                          int32_t* d_sorted_bags, int32_t* d_n_lookups, void* stream) {
    return prepare_both(ctx, pop, d_n_pop, non, d_n_non, d_sorted_slots, d_sorted_bags, d_n_lookups, false, stream);
}

extern "C" int32_t hl_embbag_bwd_prepare_merged(hl_ctx* ctx, const hl_ubatch* pop, const int32_t* d_n_pop,
                                                const hl_ubatch* non, const int32_t* d_n_non, int32_t* d_sorted_slots,
                                                int32_t* d_sorted_bags, int32_t* d_n_lookups, void* stream) {
    return prepare_both(ctx, pop, d_n_pop, non, d_n_non, d_sorted_slots, d_sorted_bags, d_n_lookups, true, stream);
}

extern "C" int32_t hl_embbag_bwd_apply2(hl_ctx* ctx, float* d_cache, const int32_t* d_sorted_slots,
                                        const int32_t* d_sorted_bags, const int32_t* d_n_lookups, int32_t which,
                                        const float* d_grad_out, float lr, void* stream_) {
    if (!ctx || !d_cache || !d_n_lookups || !d_grad_out || (which != 0 && which != 1)) return HL_EINVAL;
    if (ctx->max_nnz == 0) return HL_OK;
    if (!d_sorted_slots || !d_sorted_bags) return HL_EINVAL;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    const int32_t* d_first = which == 0 ? nullptr : d_n_lookups;             // X's block starts behind O's
    const int32_t bias = which == 0 ? 0 : (int32_t)(ctx->hot_cap + ctx->staging_cap + 1);
#define HL_BWD(G, NV) \
    launch_bwd<G, NV>(ctx, d_cache, d_sorted_slots, d_sorted_bags, d_n_lookups + which, d_grad_out, lr, stream, d_first, bias)
    HL_DISPATCH_ROW_SHAPE(ctx->D / 4, HL_BWD);
#undef HL_BWD
}

extern "C" int32_t hl_embbag_bwd_apply(hl_ctx* ctx, float* d_cache, const int32_t* d_sorted_slots,
                                       const int32_t* d_sorted_bags, const int32_t* d_n_lookups,
                                       const float* d_grad_out, float lr, void* stream_) {
    if (!ctx || !d_cache || !d_n_lookups || !d_grad_out) return HL_EINVAL;
    if (ctx->max_nnz == 0) return HL_OK;
    if (!d_sorted_slots || !d_sorted_bags) return HL_EINVAL;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
#define HL_BWD(G, NV) launch_bwd<G, NV>(ctx, d_cache, d_sorted_slots, d_sorted_bags, d_n_lookups, d_grad_out, lr, stream)
    HL_DISPATCH_ROW_SHAPE(ctx->D / 4, HL_BWD);
#undef HL_BWD
}

// ---------------------------------------------------------------------------------------------------------------
// Backward without a context or a workspace: the scratch is a fixed array inside the library image.
// ---------------------------------------------------------------------------------------------------------------
namespace hl {
namespace {

constexpr int64_t kStaticMaxNnz = HL_STATIC_MAX_NNZ;
constexpr int64_t kStaticMaxDim = HL_STATIC_MAX_DIM;

constexpr size_t align256(size_t x) { return (x + 255) & ~size_t(255); }
// layout of the static scratch: [header: status (8 ints), bag count word + lookup count (8 ints)] [keys x2]
// [vals x2] [histogram] [partial sums]
constexpr size_t kStaticHeaderBytes = 256;
constexpr size_t kStaticPairBytes = align256(size_t(kStaticMaxNnz) * sizeof(int32_t));
constexpr int64_t kStaticHistWords = sort_hist_words(kStaticMaxNnz);
constexpr size_t kStaticHistBytes = align256(size_t(kStaticHistWords) * sizeof(uint32_t));
constexpr size_t kStaticPartBytes =
    align256(size_t(2) * ((kStaticMaxNnz + kBwdChunk - 1) / kBwdChunk) * kStaticMaxDim * sizeof(float) +
             bwd_span_list_words(kStaticMaxNnz) * sizeof(int32_t));
constexpr size_t kStaticScratchBytes = kStaticHeaderBytes + 4 * kStaticPairBytes + kStaticHistBytes + kStaticPartBytes;

// Lives in every device's copy of the library image from load to exit (about 3 MB).  The name below is only a
// host-side handle for cudaGetSymbolAddress; kernels get the real device address as an argument.
static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

std::mutex g_static_mutex;
unsigned char* g_static_ptr[64] = {};   // device address of g_static_scratch, per device ordinal

__global__ void k_static_begin(int32_t* header, int32_t n_bags, int32_t* span_count) {
    header[0] = 0;        // status word: every call starts clean
    header[8] = n_bags;   // the backward kernels read their bag count from device memory
    // the count words of the backward's run list: their place in the array depends on the call's sizes, so an earlier
    // call may have left partial sums there
    for (int i = 0; i < 8; ++i) span_count[i] = 0;
}

__global__ void k_static_end(const int32_t* header, int32_t* d_status) { *d_status = header[0]; }

}  // namespace
}  // namespace hl

extern "C" int32_t hl_embbag_bwd_sgd_static(float* d_cache, int64_t cache_rows, int32_t dim,
                                            const int32_t* d_offsets, const int32_t* d_ids, int32_t n_bags,
                                            int64_t nnz, const float* d_grad_out, float lr, int32_t* d_status,
                                            void* stream_) {
    if (!d_cache || !d_offsets || !d_grad_out || cache_rows < 1 || cache_rows >= (int64_t(1) << 31) - 2)
        return HL_EINVAL;
    if (dim < 4 || (dim & 3) || n_bags < 0 || nnz < 0 || (nnz > 0 && !d_ids)) return HL_EINVAL;
    if (nnz > kStaticMaxNnz || n_bags > kStaticMaxNnz || dim > kStaticMaxDim) return HL_ECAPACITY;
    if (sort_hist_words(nnz) > kStaticHistWords) return HL_ECAPACITY;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);

    // set-up, once per device: ask the runtime where this device keeps the array
    int dev = 0;
    HL_CUDA_TRY(cudaGetDevice(&dev));
    if (dev < 0 || dev >= 64) return HL_EINVAL;
    unsigned char* base = nullptr;
    {
        std::lock_guard<std::mutex> lock(g_static_mutex);
        if (!g_static_ptr[dev]) {
            void* p = nullptr;
            if (cudaGetSymbolAddress(&p, g_static_scratch) != cudaSuccess || !p) return HL_ECUDA;
            g_static_ptr[dev] = static_cast<unsigned char*>(p);
        }
        base = g_static_ptr[dev];
    }
    if (nnz == 0 || n_bags == 0) {
        if (d_status) HL_CUDA_TRY(cudaMemsetAsync(d_status, 0, sizeof(int32_t), stream));
        return HL_OK;
    }

    // a context on the stack whose backward region points into the static array; nothing else is used
    hl_ctx tmp{};
    tmp.T = 1;
    tmp.S = 1;
    tmp.D = dim;
    tmp.N = cache_rows;
    tmp.max_batch = n_bags;
    tmp.max_bags = n_bags;
    tmp.max_nnz = nnz;
    tmp.hot_cap = cache_rows;
    tmp.staging_cap = 0;
    int32_t* header = reinterpret_cast<int32_t*>(base);
    unsigned char* p = base + kStaticHeaderBytes;
    tmp.r.status = header;
    tmp.r.bwd_n = header + 12;
    for (int i = 0; i < 2; ++i) {
        tmp.r.bwd_keys[i] = reinterpret_cast<int32_t*>(p);
        p += kStaticPairBytes;
        tmp.r.bwd_vals[i] = reinterpret_cast<int32_t*>(p);
        p += kStaticPairBytes;
    }
    tmp.r.bwd_hist = reinterpret_cast<uint32_t*>(p);
    p += kStaticHistBytes;
    tmp.r.bwd_part = reinterpret_cast<float*>(p);

    k_static_begin<<<1, 1, 0, stream>>>(header, n_bags, span_count_of(&tmp));
    note_launches(1);
    HL_LAUNCH_CHECK();
    hl_ubatch ub{const_cast<int32_t*>(d_offsets), const_cast<int32_t*>(d_ids), nnz};
    const int32_t st = hl_embbag_bwd_sgd(&tmp, d_cache, &ub, header + 8, d_grad_out, lr, stream_);
    if (st != HL_OK) return st;
    if (d_status) {
        k_static_end<<<1, 1, 0, stream>>>(header, d_status);
        note_launches(1);
        HL_LAUNCH_CHECK();
    }
    return HL_OK;
}
