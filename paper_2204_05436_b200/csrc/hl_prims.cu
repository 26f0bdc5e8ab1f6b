// Device-wide primitives used by several steps: exclusive scan and stable LSD radix sort of pairs.
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

// ---- scan ---------------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(kThreads) k_scan_tile_sums(const int32_t* __restrict__ in, const int32_t* d_n,
                                                             int64_t n_max, int32_t* __restrict__ tiles) {
    __shared__ int smem[40];
    const int64_t n = clamp_n(d_n, n_max);
    const int64_t base = (int64_t)blockIdx.x * kScanTile + (int64_t)threadIdx.x * kItems;
    int s = 0;
#pragma unroll
    for (int i = 0; i < kItems; ++i)
        if (base + i < n) s += in[base + i];
    int total;
    block_exclusive_scan(s, smem, total);
    if (threadIdx.x == 0) tiles[blockIdx.x] = total;
}

// Single block: exclusive scan of vals[0 .. count) in place, vals[count] = total.
__global__ void __launch_bounds__(1024) k_scan_spine(int32_t* __restrict__ vals, int64_t count) {
    __shared__ int smem[40];
    constexpr int kPer = 16;
    int carry = 0;
    for (int64_t start = 0; start < count; start += 1024 * kPer) {
        const int64_t base = start + (int64_t)threadIdx.x * kPer;
        int v[kPer];
        int s = 0;
#pragma unroll
        for (int i = 0; i < kPer; ++i) {
            v[i] = base + i < count ? vals[base + i] : 0;
            s += v[i];
        }
        int total;
        int excl = block_exclusive_scan(s, smem, total) + carry;
#pragma unroll
        for (int i = 0; i < kPer; ++i) {
            if (base + i < count) vals[base + i] = excl;
            excl += v[i];
        }
        carry += total;
    }
    if (threadIdx.x == 0) vals[count] = carry;
}

__global__ void __launch_bounds__(kThreads) k_scan_apply(const int32_t* in, int32_t* out, const int32_t* d_n,
                                                         int64_t n_max, const int32_t* __restrict__ tiles,
                                                         int64_t n_tiles) {
    __shared__ int smem[40];
    const int64_t n = clamp_n(d_n, n_max);
    const int64_t base = (int64_t)blockIdx.x * kScanTile + (int64_t)threadIdx.x * kItems;
    int v[kItems];
    int s = 0;
#pragma unroll
    for (int i = 0; i < kItems; ++i) {
        v[i] = base + i < n ? in[base + i] : 0;
        s += v[i];
    }
    int total;
    int excl = block_exclusive_scan(s, smem, total) + tiles[blockIdx.x];
#pragma unroll
    for (int i = 0; i < kItems; ++i) {
        if (base + i < n) out[base + i] = excl;
        excl += v[i];
    }
    if (blockIdx.x == 0 && threadIdx.x == 0) out[n] = tiles[n_tiles];
}

// ---- radix sort ---------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(kThreads) k_sort_hist(const int32_t* __restrict__ keys, const int32_t* d_n,
                                                        int64_t n_max, int shift, uint32_t* __restrict__ hist,
                                                        int64_t n_tiles) {
    __shared__ uint32_t h[256];
    h[threadIdx.x] = 0;
    __syncthreads();
    const int64_t n = clamp_n(d_n, n_max);
    const int64_t base = (int64_t)blockIdx.x * kSortTile;
#pragma unroll
    for (int i = 0; i < kItems; ++i) {
        const int64_t idx = base + (int64_t)i * kThreads + threadIdx.x;
        if (idx < n) atomicAdd(&h[((uint32_t)keys[idx] >> shift) & 255u], 1u);
    }
    __syncthreads();
    hist[(int64_t)threadIdx.x * n_tiles + blockIdx.x] = h[threadIdx.x];
}

// Stable scatter.  Order of the items of a tile: warp-major, then round, then lane.
__global__ void __launch_bounds__(kThreads) k_sort_scatter(const int32_t* __restrict__ keys_in,
                                                           const int32_t* __restrict__ vals_in,
                                                           int32_t* __restrict__ keys_out,
                                                           int32_t* __restrict__ vals_out, const int32_t* d_n,
                                                           int64_t n_max, int shift,
                                                           const uint32_t* __restrict__ hist, int64_t n_tiles) {
    constexpr int kWarps = kThreads / 32;
    __shared__ uint32_t cnt[kWarps][256];
    __shared__ uint32_t digit_base[256];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    for (int i = threadIdx.x; i < kWarps * 256; i += kThreads) (&cnt[0][0])[i] = 0;
    __syncthreads();

    const int64_t n = clamp_n(d_n, n_max);
    const int64_t warp_base = (int64_t)blockIdx.x * kSortTile + (int64_t)warp * (32 * kItems);
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
    {   // one thread per digit: exclusive prefix over the warps, plus this tile's global base for the digit
        const int d = threadIdx.x;
        uint32_t run = 0;
#pragma unroll
        for (int w = 0; w < kWarps; ++w) {
            const uint32_t c = cnt[w][d];
            cnt[w][d] = run;
            run += c;
        }
        digit_base[d] = hist[(int64_t)d * n_tiles + blockIdx.x];
    }
    __syncthreads();
#pragma unroll
    for (int r = 0; r < kItems; ++r) {
        const int64_t idx = warp_base + r * 32 + lane;
        if (idx < n) {
            const uint32_t d = ((uint32_t)key[r] >> shift) & 255u;
            const int64_t pos = (int64_t)digit_base[d] + cnt[warp][d] + rank[r];
            keys_out[pos] = key[r];
            vals_out[pos] = val[r];
        }
    }
}

}  // namespace

int32_t exclusive_scan_i32(const int32_t* in, int32_t* out, const int32_t* d_n, int64_t n_max, int32_t* tiles,
                           cudaStream_t stream) {
    if (n_max <= 0) {
        HL_CUDA_TRY(cudaMemsetAsync(out, 0, sizeof(int32_t), stream));
        return HL_OK;
    }
    const int64_t n_tiles = div_up(n_max, kScanTile);
    k_scan_tile_sums<<<(unsigned)n_tiles, kThreads, 0, stream>>>(in, d_n, n_max, tiles);
    k_scan_spine<<<1, 1024, 0, stream>>>(tiles, n_tiles);
    k_scan_apply<<<(unsigned)n_tiles, kThreads, 0, stream>>>(in, out, d_n, n_max, tiles, n_tiles);
    note_launches(3);
    HL_LAUNCH_CHECK();
    return HL_OK;
}

int32_t radix_sort_pairs(int32_t* keys[2], int32_t* vals[2], const int32_t* d_n, int64_t n_max, int key_bits,
                         uint32_t* hist, int32_t** out_keys, int32_t** out_vals, cudaStream_t stream) {
    int cur = 0;
    if (n_max > 0) {
        const int64_t n_tiles = div_up(n_max, kSortTile);
        const int64_t n_hist = 256 * n_tiles;
        const int passes = (key_bits + 7) / 8;
        for (int p = 0; p < passes; ++p) {
            const int shift = 8 * p;
            k_sort_hist<<<(unsigned)n_tiles, kThreads, 0, stream>>>(keys[cur], d_n, n_max, shift, hist, n_tiles);
            if (n_hist <= 65536) {
                k_scan_spine<<<1, 1024, 0, stream>>>(reinterpret_cast<int32_t*>(hist), n_hist);
                note_launches(1);
            } else {
                // the scan's tile sums live right behind the histogram (the workspace reserves the room)
                int32_t* tiles = reinterpret_cast<int32_t*>(hist) + n_hist + 1;
                int32_t st = exclusive_scan_i32(reinterpret_cast<int32_t*>(hist), reinterpret_cast<int32_t*>(hist),
                                                nullptr, n_hist, tiles, stream);
                if (st != HL_OK) return st;
            }
            k_sort_scatter<<<(unsigned)n_tiles, kThreads, 0, stream>>>(keys[cur], vals[cur], keys[cur ^ 1],
                                                                      vals[cur ^ 1], d_n, n_max, shift, hist,
                                                                      n_tiles);
            note_launches(2);   // histogram + scatter
            cur ^= 1;
        }
        HL_LAUNCH_CHECK();
    }
    *out_keys = keys[cur];
    *out_vals = vals[cur];
    return HL_OK;
}

}  // namespace hl
