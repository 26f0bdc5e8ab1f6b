// Device-wide primitives used by several steps: single-pass exclusive scan and stable LSD radix sort of pairs
// (one kernel per digit; tiles chained through status words instead of a separate scan of tile histograms).
// Both take their element count from device memory, so that no step has to synchronise the host.
#include <atomic>

#include "hl_common.cuh"

namespace hl {

static std::atomic<unsigned long long> g_launches{0};
void note_launches(int n) { g_launches.fetch_add((unsigned long long)n, std::memory_order_relaxed); }
unsigned long long launches_so_far() { return g_launches.load(std::memory_order_relaxed); }

namespace {

constexpr int kThreads = 256;
constexpr int kItems = 8;   // kThreads * kItems == kScanTile == kSortTile
static_assert(kThreads * kItems == kScanTile && kThreads * kItems == kSortTile, "tile shape");

__device__ __forceinline__ int warp_inclusive_scan(int v) {
    const int lane = threadIdx.x & 31;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
        int o = __shfl_up_sync(0xffffffffu, v, d);
        if (lane >= d) v += o;
    }
    return v;
}

// Exclusive scan of one value per thread over the block; `total` is the block sum (same in all threads).
// smem: at least blockDim.x / 32 + 1 ints.  Ends with a barrier, so smem can be reused right away.
__device__ __forceinline__ int block_exclusive_scan(int v, int* smem, int& total) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, n_warps = blockDim.x >> 5;
    const int incl = warp_inclusive_scan(v);
    if (lane == 31) smem[warp] = incl;
    __syncthreads();
    if (warp == 0) {
        int w = lane < n_warps ? smem[lane] : 0;
        int wi = warp_inclusive_scan(w);
        if (lane < n_warps) smem[lane] = wi - w;
        if (lane == 31) smem[32] = wi;
    }
    __syncthreads();
    const int res = smem[warp] + incl - v;
    total = smem[32];
    __syncthreads();
    return res;
}

__device__ __forceinline__ int64_t clamp_n(const int32_t* d_n, int64_t n_max) {
    if (d_n == nullptr) return n_max;
    int64_t n = *d_n;
    if (n < 0) n = 0;
    return n < n_max ? n : n_max;
}

// ---- single-pass chaining between tiles --------------------------------------------------------------------
// Tiles are handed out by a ticket counter, so a tile's predecessors are always held by blocks that have
// started.  A tile first publishes its own sum (AGGREGATE), then walks back over its predecessors adding their
// sums until it meets one that already knows its inclusive prefix (PREFIX), and finally publishes its own
// prefix.  Publishing never waits on anything, so the walk always terminates; every poll is bounded all the same,
// and a poll that runs out records HL_ETIMEOUT and carries on with what it has (positions are range-checked).
constexpr uint32_t kFlagAgg = 1u << 30, kFlagPrefix = 1u << 31, kValueMask = kFlagAgg - 1u;
constexpr unsigned long long kFlagAgg64 = 1ull << 62, kFlagPrefix64 = 1ull << 63, kValueMask64 = kFlagAgg64 - 1ull;

__device__ __forceinline__ uint32_t ld_relaxed(const uint32_t* p) {
    uint32_t v;
    asm volatile("ld.relaxed.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ void st_relaxed(uint32_t* p, uint32_t v) {
    asm volatile("st.relaxed.gpu.global.u32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}
__device__ __forceinline__ unsigned long long ld_relaxed64(const unsigned long long* p) {
    unsigned long long v;
    asm volatile("ld.relaxed.gpu.global.u64 %0, [%1];" : "=l"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ void st_relaxed64(unsigned long long* p, unsigned long long v) {
    asm volatile("st.relaxed.gpu.global.u64 [%0], %1;" ::"l"(p), "l"(v) : "memory");
}

// ---- scan ---------------------------------------------------------------------------------------------------
// st[0] = ticket counter, st[1 + tile] = status word of the tile; all zero on entry.
// max_polls / stall_tile: see WaitCfg (a stalled tile publishes nothing, so that its successors' waits run out).
__global__ void __launch_bounds__(kThreads) k_scan_chained(const int32_t* in, int32_t* out, const int32_t* d_n,
                                                           int64_t n_max, unsigned long long* st, int32_t* status,
                                                           int max_polls, int64_t stall_tile) {
    __shared__ int smem[40];
    __shared__ long long s_tile, s_excl;
    if (threadIdx.x == 0) s_tile = (long long)atomicAdd(&st[0], 1ull);
    __syncthreads();
    const int64_t tile = s_tile;
    const int64_t n = clamp_n(d_n, n_max);
    const int64_t tile_base = tile * kScanTile;
    if (tile_base > n) return;   // the tile at tile_base == n has no element but still writes out[n]
    const int64_t base = tile_base + (int64_t)threadIdx.x * kItems;
    int v[kItems];
    int s = 0;
#pragma unroll
    for (int i = 0; i < kItems; ++i) {
        v[i] = base + i < n ? in[base + i] : 0;
        s += v[i];
    }
    int total;
    int excl = block_exclusive_scan(s, smem, total);
    if (threadIdx.x < 32) {
        // warp 0 walks back over the predecessors 32 tiles at a time: lane l looks at tile t0 - l; the sums up to
        // and including the nearest tile that already knows its inclusive prefix are added
        const int lane = threadIdx.x;
        long long before = 0;
        if (tile > 0) {
            if (lane == 0 && tile != stall_tile) st_relaxed64(&st[1 + tile], kFlagAgg64 | (unsigned long long)total);
            bool done = false;
            for (int64_t t0 = tile - 1; t0 >= 0 && !done; t0 -= 32) {
                const int64_t t = t0 - lane;
                unsigned long long w = kFlagPrefix64;            // before tile 0: an empty prefix
                if (t >= 0) {
                    int polls = 0;
                    while (((w = ld_relaxed64(&st[1 + t])) & (kFlagAgg64 | kFlagPrefix64)) == 0) {
                        if (++polls > max_polls) {               // give up: carry on with what there is
                            set_status(status, HL_ETIMEOUT);
                            w = kFlagPrefix64;
                            break;
                        }
                        __nanosleep(20);
                    }
                }
                const unsigned with_prefix = __ballot_sync(0xffffffffu, (w & kFlagPrefix64) != 0);
                const int stop = with_prefix ? __ffs(with_prefix) - 1 : 31;
                long long val = lane <= stop ? (long long)(w & kValueMask64) : 0;
#pragma unroll
                for (int d = 16; d > 0; d >>= 1) val += __shfl_down_sync(0xffffffffu, val, d);
                before += __shfl_sync(0xffffffffu, val, 0);
                done = with_prefix != 0;
            }
        }
        if (lane == 0) {
            if (tile != stall_tile) st_relaxed64(&st[1 + tile], kFlagPrefix64 | (unsigned long long)(before + total));
            s_excl = before;
            if (n < tile_base + kScanTile) out[n] = (int32_t)(before + total);
        }
    }
    __syncthreads();
    excl += (int)s_excl;
#pragma unroll
    for (int i = 0; i < kItems; ++i) {
        if (base + i < n) out[base + i] = excl;
        excl += v[i];
    }
}

// ---- radix sort ---------------------------------------------------------------------------------------------
// Digit histograms of all passes in one sweep over the keys.
__global__ void __launch_bounds__(kThreads) k_sort_digit_hist(const int32_t* __restrict__ keys, const int32_t* d_n,
                                                              int64_t n_max, int passes,
                                                              uint32_t* __restrict__ ghist /* [passes][256] */) {
    __shared__ uint32_t h[4][256];
    for (int i = threadIdx.x; i < 4 * 256; i += kThreads) (&h[0][0])[i] = 0;
    __syncthreads();
    const int64_t n = clamp_n(d_n, n_max);
    for (int64_t i = (int64_t)blockIdx.x * kThreads + threadIdx.x; i < n; i += (int64_t)gridDim.x * kThreads) {
        const uint32_t k = (uint32_t)keys[i];
        for (int p = 0; p < passes; ++p) atomicAdd(&h[p][(k >> (8 * p)) & 255u], 1u);
    }
    __syncthreads();
    for (int i = threadIdx.x; i < passes * 256; i += kThreads) {
        const uint32_t c = (&h[0][0])[i];
        if (c) atomicAdd(&ghist[i], c);
    }
}

// One pass: stable scatter by one digit.  Order of the items of a tile: warp-major, then round, then lane.
// ghist: this pass's 256 digit counts; ticket: tile counter; tstat[tile][256]: status words, zero on entry.
__global__ void __launch_bounds__(kThreads) k_sort_pass(const int32_t* __restrict__ keys_in,
                                                        const int32_t* __restrict__ vals_in,
                                                        int32_t* __restrict__ keys_out, int32_t* __restrict__ vals_out,
                                                        const int32_t* d_n, int64_t n_max, int shift,
                                                        const uint32_t* __restrict__ ghist, uint32_t* ticket,
                                                        uint32_t* tstat, int32_t* status, int max_polls,
                                                        int64_t stall_tile) {
    constexpr int kWarps = kThreads / 32;
    __shared__ uint32_t cnt[kWarps][256];
    __shared__ uint32_t digit_base[256];
    __shared__ int scan_smem[40];
    __shared__ uint32_t s_tile;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    if (threadIdx.x == 0) s_tile = atomicAdd(ticket, 1u);
    for (int i = threadIdx.x; i < kWarps * 256; i += kThreads) (&cnt[0][0])[i] = 0;
    __syncthreads();
    const int64_t tile = s_tile;
    const int64_t n = clamp_n(d_n, n_max);
    if (tile * kSortTile >= n) return;

    const int64_t warp_base = tile * kSortTile + (int64_t)warp * (32 * kItems);
    int32_t key[kItems], val[kItems];
    uint32_t rank[kItems];
    const unsigned lt = lanemask_lt();
#pragma unroll
    for (int r = 0; r < kItems; ++r) {
        const int64_t idx = warp_base + r * 32 + lane;
        const bool valid = idx < n;
        key[r] = valid ? keys_in[idx] : 0;
        val[r] = valid ? vals_in[idx] : 0;
        const uint32_t d = valid ? (((uint32_t)key[r] >> shift) & 255u) : 256u;
        const unsigned peers = __match_any_sync(0xffffffffu, d);
        uint32_t before = 0;
        if (valid) before = cnt[warp][d];
        __syncwarp();
        rank[r] = before + __popc(peers & lt);
        if (valid && (peers & lt) == 0) cnt[warp][d] = before + __popc(peers);
        __syncwarp();
    }
    __syncthreads();
    // one thread per digit: prefix over the warps; then chain with the earlier tiles
    const int d = threadIdx.x;
    uint32_t total = 0;
#pragma unroll
    for (int w = 0; w < kWarps; ++w) {
        const uint32_t c = cnt[w][d];
        cnt[w][d] = total;
        total += c;
    }
    uint32_t before = 0;
    uint32_t* my = tstat + tile * 256 + d;
    if (tile > 0) {
        if (tile != stall_tile) st_relaxed(my, kFlagAgg | total);
        // walk back kLook tiles at a time (32 at a time was no faster and cost 16 registers): the kLook status
        // words are requested together, then consumed from the
        // nearest tile outwards until one of them already carries an inclusive prefix
        constexpr int kLook = 8;
        bool found = false, gave_up = false;
        for (int64_t t0 = tile - 1; t0 >= 0 && !found && !gave_up; t0 -= kLook) {
            uint32_t w[kLook];
#pragma unroll
            for (int k = 0; k < kLook; ++k) w[k] = t0 - k >= 0 ? ld_relaxed(tstat + (t0 - k) * 256 + d) : kFlagPrefix;
#pragma unroll
            for (int k = 0; k < kLook; ++k) {
                if (found || gave_up) break;
                int polls = 0;
                while ((w[k] & (kFlagAgg | kFlagPrefix)) == 0) {
                    if (++polls > max_polls) {
                        set_status(status, HL_ETIMEOUT);
                        gave_up = true;
                        break;
                    }
                    __nanosleep(20);
                    w[k] = ld_relaxed(tstat + (t0 - k) * 256 + d);
                }
                before += w[k] & kValueMask;
                found = (w[k] & kFlagPrefix) != 0;
            }
        }
    }
    if (tile != stall_tile) st_relaxed(my, kFlagPrefix | ((before + total) & kValueMask));
    int all;
    const int gbase = block_exclusive_scan((int)ghist[d], scan_smem, all);   // keys with a smaller digit
    digit_base[d] = (uint32_t)gbase + before;
    __syncthreads();
#pragma unroll
    for (int r = 0; r < kItems; ++r) {
        const int64_t idx = warp_base + r * 32 + lane;
        if (idx < n) {
            const uint32_t dg = ((uint32_t)key[r] >> shift) & 255u;
            const int64_t pos = (int64_t)digit_base[dg] + cnt[warp][dg] + rank[r];
            if (pos < n) {   // always true unless a chain poll gave up
                keys_out[pos] = key[r];
                vals_out[pos] = val[r];
            }
        }
    }
}

__global__ void __launch_bounds__(kThreads) k_zero_words(uint32_t* p, int64_t n) {
    for (int64_t i = (int64_t)blockIdx.x * kThreads + threadIdx.x; i < n; i += (int64_t)gridDim.x * kThreads) p[i] = 0u;
}

}  // namespace

// ---- the same two primitives, launched from the device --------------------------------------------------------
// For a kernel that learns on the device that follow-up work is needed (the cold-row search beyond its one-cluster
// path): ONE thread calls these; every launch goes to the tail-launch stream of the calling grid, i.e. runs after
// that grid has finished, one launch after the other, before anything the host queued behind the grid.  n is known
// here, so the grids are exact.  A launch the device runtime refuses sets HL_ECUDA in *status.
__device__ static void tail_check(int32_t* status) {
    if (cudaGetLastError() != cudaSuccess) set_status(status, HL_ECUDA);
}

__device__ int radix_sort_pairs_tail(int32_t* keys0, int32_t* keys1, int32_t* vals0, int32_t* vals1, int64_t n,
                                     int key_bits, uint32_t* hist, int32_t* status, int max_polls) {
    if (n <= 0) return 0;
    const int64_t n_tiles = (n + kSortTile - 1) / kSortTile;
    const int passes = (key_bits + 7) / 8;
    uint32_t* ghist = hist;
    uint32_t* ticket = hist + 4 * 256;
    uint32_t* tstat = hist + 4 * 256 + 8;
    const int64_t words = 4 * 256 + 8 + (int64_t)passes * n_tiles * 256;
    int64_t zero_grid = (words + kThreads * 8 - 1) / (kThreads * 8);
    k_zero_words<<<(unsigned)(zero_grid < 1024 ? zero_grid : 1024), kThreads, 0, cudaStreamTailLaunch>>>(hist, words);
    int64_t hist_grid = (n + kThreads * 8 - 1) / (kThreads * 8);
    k_sort_digit_hist<<<(unsigned)hist_grid, kThreads, 0, cudaStreamTailLaunch>>>(keys0, nullptr, n, passes, ghist);
    int32_t* k[2] = {keys0, keys1};
    int32_t* v[2] = {vals0, vals1};
    int cur = 0;
    for (int p = 0; p < passes; ++p) {
        k_sort_pass<<<(unsigned)n_tiles, kThreads, 0, cudaStreamTailLaunch>>>(
            k[cur], v[cur], k[cur ^ 1], v[cur ^ 1], nullptr, n, 8 * p, ghist + 256 * p, ticket + p,
            tstat + (size_t)p * n_tiles * 256, status, max_polls, (int64_t)-1);
        cur ^= 1;
    }
    tail_check(status);
    return cur;
}

__device__ void exclusive_scan_i32_tail(const int32_t* in, int32_t* out, int64_t n, int32_t* tiles, int32_t* status,
                                        int max_polls) {
    const int64_t n_tiles = n / kScanTile + 1;
    k_zero_words<<<1, kThreads, 0, cudaStreamTailLaunch>>>(reinterpret_cast<uint32_t*>(tiles), 2 * (n_tiles + 1));
    k_scan_chained<<<(unsigned)n_tiles, kThreads, 0, cudaStreamTailLaunch>>>(
        in, out, nullptr, n, reinterpret_cast<unsigned long long*>(tiles), status, max_polls, (int64_t)-1);
    tail_check(status);
}

int32_t exclusive_scan_i32(const int32_t* in, int32_t* out, const int32_t* d_n, int64_t n_max, int32_t* tiles,
                           int32_t* status, cudaStream_t stream, WaitCfg w) {
    if (n_max <= 0) {
        HL_CUDA_TRY(cudaMemsetAsync(out, 0, sizeof(int32_t), stream));
        return HL_OK;
    }
    const int64_t n_tiles = n_max / kScanTile + 1;   // one more than needed when n is a multiple of the tile
    unsigned long long* st = reinterpret_cast<unsigned long long*>(tiles);
    HL_CUDA_TRY(cudaMemsetAsync(st, 0, sizeof(unsigned long long) * (n_tiles + 1), stream));
    k_scan_chained<<<(unsigned)n_tiles, kThreads, 0, stream>>>(in, out, d_n, n_max, st, status, w.max_polls,
                                                               w.stall_tile);
    note_launches(1);
    HL_LAUNCH_CHECK();
    return HL_OK;
}

int32_t radix_sort_pairs(int32_t* keys[2], int32_t* vals[2], const int32_t* d_n, int64_t n_max, int key_bits,
                         uint32_t* hist, int32_t* status, int32_t** out_keys, int32_t** out_vals,
                         cudaStream_t stream, WaitCfg w) {
    int cur = 0;
    if (n_max > 0) {
        const int64_t n_tiles = div_up(n_max, kSortTile);
        const int passes = (key_bits + 7) / 8;
        if (passes > 4) return HL_EINVAL;
        // scratch: [4][256] digit counts, 8 ticket words, [4][n_tiles][256] tile status words
        uint32_t* ghist = hist;
        uint32_t* ticket = hist + 4 * 256;
        uint32_t* tstat = hist + 4 * 256 + 8;
        HL_CUDA_TRY(cudaMemsetAsync(hist, 0, sizeof(uint32_t) * (4 * 256 + 8 + (size_t)passes * n_tiles * 256),
                                    stream));
        k_sort_digit_hist<<<grid_for(n_max, kThreads * 8, 1024), kThreads, 0, stream>>>(keys[0], d_n, n_max,
                                                                                            passes, ghist);
        for (int p = 0; p < passes; ++p) {
            k_sort_pass<<<(unsigned)n_tiles, kThreads, 0, stream>>>(keys[cur], vals[cur], keys[cur ^ 1], vals[cur ^ 1],
                                                                    d_n, n_max, 8 * p, ghist + 256 * p, ticket + p,
                                                                    tstat + (size_t)p * n_tiles * 256, status,
                                                                    w.max_polls, w.stall_tile);
            cur ^= 1;
        }
        note_launches(1 + passes);
        HL_LAUNCH_CHECK();
    }
    *out_keys = keys[cur];
    *out_vals = vals[cur];
    return HL_OK;
}

}  // namespace hl
