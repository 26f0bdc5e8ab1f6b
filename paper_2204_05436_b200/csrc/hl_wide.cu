// The index-only calls of the path for models with 2^31 rows and more (the paper's SYN-M1/M2 sizes): global row ids
// are 64-bit, counted in a hashed counter and looked up in a hashed remap whose hash is the randomizer of Section
// V-C.  Every table still has fewer than 2^31 rows, so a row is the pair (table, table-local index): the order of
// global ids is the order of those pairs, which two stable 32-bit sorts give (index, then table).
#include <stdlib.h>

#include "hl_common.cuh"

namespace hl {
namespace {

constexpr int kThreads = 256;

struct Carver {
    char* base;
    size_t off = 0;
    template <typename T>
    T* take(int64_t count) {
        off = (off + 255) & ~size_t(255);
        T* p = base ? reinterpret_cast<T*>(base + off) : nullptr;
        off += (size_t)count * sizeof(T);
        return p;
    }
};

int64_t pow2_at_least(int64_t x) {
    int64_t p = 1;
    while (p < x) p <<= 1;
    return p;
}

int bits_for(int64_t max_value) {
    int b = 1;
    while ((int64_t(1) << b) <= max_value) ++b;
    return b;
}

size_t carve(char* base, hl_wide* w) {
    Carver c{base};
    const int64_t nnz = w->max_nnz > 0 ? w->max_nnz : 1;
    const int64_t E = w->counter_slots;
    const int64_t sort_n = E > nnz ? E : nnz;
    w->status = c.take<int32_t>(8);
    w->table_base = c.take<int64_t>(w->T + 1);
    w->c_keys = c.take<long long>(E);
    w->c_cnt = c.take<uint32_t>(E);
    w->sel = c.take<SelectState>(1);
    w->sel_gt = c.take<uint32_t>(div_up(E, kSelTile) + 2);
    w->sel_eq = c.take<uint32_t>(div_up(E, kSelTile) + 2);
    w->n_seen = c.take<int32_t>(4);
    w->e_tab = c.take<int32_t>(E);
    w->e_idx = c.take<int32_t>(E);
    w->e_cnt = c.take<uint32_t>(E);
    w->s_cnt = c.take<uint32_t>(E);
    w->s_ent = c.take<int32_t>(E);
    w->sel_idx = c.take<int32_t>(w->hot_cap > 0 ? w->hot_cap : 1);
    w->r_keys = c.take<long long>(w->remap_slots);
    w->r_vals = c.take<int32_t>(w->remap_slots);
    for (int i = 0; i < 2; ++i) {
        w->sort_keys[i] = c.take<int32_t>(sort_n);
        w->sort_vals[i] = c.take<int32_t>(sort_n);
    }
    w->sort_hist = c.take<uint32_t>(sort_hist_words(sort_n));
    w->frag_flags = c.take<uint8_t>(w->max_batch);
    w->frag_scan = c.take<int32_t>(w->max_bags + 2);
    w->frag_tiles = c.take<int32_t>(scan_tile_words(w->max_bags));
    w->cold_tab = c.take<int32_t>(nnz);
    w->cold_idx = c.take<int32_t>(nnz);
    w->cold_pos = c.take<int32_t>(nnz);
    w->cold_rank = c.take<int32_t>(nnz + 2);
    w->cold_tiles = c.take<int32_t>(scan_tile_words(nnz));
    w->cold_n = c.take<int32_t>(4);
    return (c.off + 255) & ~size_t(255);
}

bool fill(hl_wide* w, const hl_geometry* g, int32_t max_batch, int64_t max_nnz, int64_t hot_cap, int64_t staging_cap,
          int64_t counter_slots) {
    if (!g || g->num_tables < 1 || g->num_tables > 255 || g->bags_per_sample < 1 || !g->table_rows) return false;
    if (max_batch < 1 || max_nnz < 0 || hot_cap < 0 || staging_cap < 0 || counter_slots < 2) return false;
    int64_t n = 0;
    for (int t = 0; t < g->num_tables; ++t) {
        if (g->table_rows[t] < 1 || g->table_rows[t] >= (int64_t(1) << 31)) return false;   // table-local ids are int32
        n += g->table_rows[t];
        if (n >= (int64_t(1) << 56)) return false;
    }
    w->T = g->num_tables;
    w->S = g->bags_per_sample;
    w->N = n;
    w->max_batch = max_batch;
    w->max_nnz = max_nnz;
    w->max_bags = (int64_t)g->num_tables * max_batch * g->bags_per_sample;
    w->hot_cap = hot_cap;
    w->staging_cap = staging_cap;
    w->counter_slots = pow2_at_least(counter_slots);
    w->remap_slots = pow2_at_least(2 * (hot_cap > 0 ? hot_cap : 1));
    if (w->max_bags >= (int64_t(1) << 30) || max_nnz >= (int64_t(1) << 30) || w->counter_slots >= (int64_t(1) << 30) ||
        hot_cap + staging_cap >= (int64_t(1) << 31) - 2)
        return false;
    return true;
}

// ---- hashed counter ---------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(kThreads) k_wide_count(const int32_t* __restrict__ indices,
                                                         const int32_t* __restrict__ offsets, int64_t n_bags,
                                                         int64_t bags_per_table, const int64_t* __restrict__ table_base,
                                                         long long* keys, uint32_t* cnt, uint64_t mask,
                                                         SelectState* sel, int32_t* status) {
    unsigned long long mine = 0;
    for (int64_t bag = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; bag < n_bags;
         bag += (int64_t)gridDim.x * blockDim.x) {
        const int t = (int)(bag / bags_per_table);
        const int64_t base = table_base[t], rows = table_base[t + 1] - base;
        for (int32_t j = offsets[bag]; j < offsets[bag + 1]; ++j) {
            const int32_t idx = indices[j];
            if (idx < 0 || idx >= rows) {
                set_status(status, HL_EBOUNDS);
                continue;
            }
            const long long g = base + idx;
            uint64_t h = randomize64((uint64_t)g) & mask;
            bool placed = false;
            for (uint64_t tries = 0; tries <= mask; ++tries) {     // linear probing; the first free entry is claimed
                long long k = keys[h];
                if (k < 0) k = (long long)atomicCAS(reinterpret_cast<unsigned long long*>(&keys[h]),
                                                    (unsigned long long)-1LL, (unsigned long long)g);
                if (k < 0 || k == g) {
                    atomicAdd(&cnt[h], 1u);
                    placed = true;
                    break;
                }
                h = (h + 1) & mask;
            }
            if (!placed) set_status(status, HL_ECAPACITY);         // more distinct rows than the counter holds
            else ++mine;
        }
    }
#pragma unroll
    for (int d = 16; d > 0; d >>= 1) mine += __shfl_down_sync(0xffffffffu, mine, d);
    if ((threadIdx.x & 31) == 0 && mine) atomicAdd(&sel->total, mine);
}

// every counted row as (table, index, count), in no particular order
__global__ void __launch_bounds__(kThreads) k_wide_entries(const long long* __restrict__ keys,
                                                           const uint32_t* __restrict__ cnt, int64_t slots,
                                                           const int64_t* __restrict__ table_base, int T,
                                                           int32_t* n_seen, int32_t* e_tab, int32_t* e_idx,
                                                           uint32_t* e_cnt, int32_t* sort_key, int32_t* sort_val) {
    for (int64_t h = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; h < slots; h += (int64_t)gridDim.x * blockDim.x) {
        const long long g = keys[h];
        if (g < 0) continue;
        int lo = 0, hi = T;                      // table_base[lo] <= g < table_base[hi]
        while (hi - lo > 1) {
            const int mid = (lo + hi) >> 1;
            if (table_base[mid] <= g) lo = mid;
            else hi = mid;
        }
        const int32_t i = atomicAdd(n_seen, 1);
        e_tab[i] = lo;
        e_idx[i] = (int32_t)(g - table_base[lo]);
        e_cnt[i] = cnt[h];
        sort_key[i] = e_idx[i];
        sort_val[i] = i;
    }
}

// out_key[j] = table[val[j]]: the key of the second, stable sort
__global__ void __launch_bounds__(kThreads) k_wide_gather_key(const int32_t* __restrict__ val,
                                                              const int32_t* __restrict__ table, const int32_t* d_n,
                                                              int64_t n_max, int32_t* __restrict__ out_key) {
    int64_t n = *d_n;
    n = n < n_max ? n : n_max;
    for (int64_t j = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; j < n; j += (int64_t)gridDim.x * blockDim.x)
        out_key[j] = table[val[j]];
}

// counts in row order (zero behind the last counted row), and the entry behind every position
__global__ void __launch_bounds__(kThreads) k_wide_row_order(const int32_t* __restrict__ val,
                                                             const uint32_t* __restrict__ e_cnt, const int32_t* d_n,
                                                             int64_t n_max, uint32_t* __restrict__ s_cnt,
                                                             int32_t* __restrict__ s_ent) {
    int64_t n = *d_n;
    n = n < n_max ? n : n_max;
    for (int64_t j = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; j < n_max; j += (int64_t)gridDim.x * blockDim.x) {
        s_cnt[j] = j < n ? e_cnt[val[j]] : 0u;
        s_ent[j] = j < n ? val[j] : -1;
    }
}

__global__ void __launch_bounds__(kThreads) k_wide_hot_rows(const int32_t* __restrict__ sel_idx,
                                                            const int64_t* __restrict__ d_n_hot, int64_t hot_cap,
                                                            const int32_t* __restrict__ s_ent,
                                                            const int32_t* __restrict__ e_tab,
                                                            const int32_t* __restrict__ e_idx,
                                                            const int64_t* __restrict__ table_base,
                                                            long long* __restrict__ hot_rows) {
    int64_t n = *d_n_hot;
    n = n < hot_cap ? n : hot_cap;
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (int64_t)gridDim.x * blockDim.x) {
        const int32_t e = s_ent[sel_idx[i]];
        hot_rows[i] = table_base[e_tab[e]] + e_idx[e];
    }
}

// ---- hashed remap -----------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(kThreads) k_wide_remap(const long long* __restrict__ hot_rows,
                                                         const int64_t* __restrict__ d_n_hot, int64_t hot_cap,
                                                         int64_t N, long long* keys, int32_t* vals, uint64_t mask,
                                                         int32_t* status) {
    int64_t n = *d_n_hot;
    if (n > hot_cap) {
        if (blockIdx.x == 0 && threadIdx.x == 0) set_status(status, HL_ECAPACITY);
        n = hot_cap;
    }
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (int64_t)gridDim.x * blockDim.x) {
        const long long g = hot_rows[i];
        if (g < 0 || g >= N || (i > 0 && hot_rows[i - 1] >= g)) {   // must be strictly ascending, in range
            set_status(status, HL_EINVAL);
            continue;
        }
        uint64_t h = randomize64((uint64_t)g) & mask;
        for (uint64_t tries = 0; tries <= mask; ++tries) {
            const long long k = (long long)atomicCAS(reinterpret_cast<unsigned long long*>(&keys[h]),
                                                     (unsigned long long)-1LL, (unsigned long long)g);
            if (k < 0) {
                vals[h] = (int32_t)i;              // the slot of a popular row is its rank in the ascending list
                break;
            }
            h = (h + 1) & mask;
        }
    }
}

}  // namespace
}  // namespace hl

using namespace hl;

extern "C" size_t hl_wide_workspace_bytes(const hl_geometry* geom, int32_t max_batch, int64_t max_nnz,
                                          int64_t hot_cap_rows, int64_t staging_cap_rows, int64_t counter_slots) {
    hl_wide w{};
    if (!fill(&w, geom, max_batch, max_nnz, hot_cap_rows, staging_cap_rows, counter_slots)) return 0;
    return carve(nullptr, &w);
}

extern "C" int32_t hl_wide_create(hl_wide** out, const hl_geometry* geom, int32_t max_batch, int64_t max_nnz,
                                  int64_t hot_cap_rows, int64_t staging_cap_rows, int64_t counter_slots,
                                  void* d_workspace, size_t ws_bytes) {
    if (!out) return HL_EINVAL;
    *out = nullptr;
    if (!d_workspace || (reinterpret_cast<uintptr_t>(d_workspace) & 255)) return HL_EINVAL;
    hl_wide* w = static_cast<hl_wide*>(calloc(1, sizeof(hl_wide)));
    if (!w) return HL_EINVAL;
    if (!fill(w, geom, max_batch, max_nnz, hot_cap_rows, staging_cap_rows, counter_slots)) {
        free(w);
        return HL_EINVAL;
    }
    if (carve(static_cast<char*>(d_workspace), w) > ws_bytes) {
        free(w);
        return HL_ECAPACITY;
    }
    int dev = 0;
    w->h_table_base = static_cast<int64_t*>(malloc(sizeof(int64_t) * (w->T + 1)));
    if (!w->h_table_base || cudaGetDevice(&dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&w->sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) {
        free(w->h_table_base);
        free(w);
        return HL_ECUDA;
    }
    w->h_table_base[0] = 0;
    for (int t = 0; t < w->T; ++t) w->h_table_base[t + 1] = w->h_table_base[t] + geom->table_rows[t];
    cudaError_t e = cudaMemcpy(w->table_base, w->h_table_base, sizeof(int64_t) * (w->T + 1), cudaMemcpyHostToDevice);
    if (e == cudaSuccess) e = cudaMemset(w->status, 0, 8 * sizeof(int32_t));
    if (e == cudaSuccess) e = cudaMemset(w->c_keys, 0xff, sizeof(long long) * w->counter_slots);
    if (e == cudaSuccess) e = cudaMemset(w->c_cnt, 0, sizeof(uint32_t) * w->counter_slots);
    if (e == cudaSuccess) e = cudaMemset(w->r_keys, 0xff, sizeof(long long) * w->remap_slots);
    if (e == cudaSuccess) e = cudaMemset(w->sel, 0, sizeof(SelectState));
    if (e == cudaSuccess) e = cudaMemset(w->frag_tiles, 0, sizeof(int32_t) * scan_tile_words(w->max_bags));
    if (e == cudaSuccess) e = cudaDeviceSynchronize();
    if (e != cudaSuccess) {
        free(w->h_table_base);
        free(w);
        return HL_ECUDA;
    }
    *out = w;
    return HL_OK;
}

extern "C" int32_t hl_wide_destroy(hl_wide* w) {
    if (!w) return HL_EINVAL;
    free(w->h_table_base);
    free(w);
    return HL_OK;
}

extern "C" int32_t hl_wide_status(hl_wide* w) {
    if (!w) return HL_EINVAL;
    HL_CUDA_TRY(cudaDeviceSynchronize());
    int32_t st = 0;
    HL_CUDA_TRY(cudaMemcpy(&st, w->status, sizeof(int32_t), cudaMemcpyDeviceToHost));
    if (st != 0) HL_CUDA_TRY(cudaMemset(w->status, 0, sizeof(int32_t)));
    return st;
}

namespace hl {
namespace {

// Sorts the pairs in sort_keys[0] / sort_vals[0] (n = *d_n of them; keys = table-local indices, values = entry numbers)
// by (table, index): a stable sort by index, then a stable sort by the tables gathered through the values.  Returns
// which buffer holds the result in *out_vals (the entry numbers in row order).
int32_t sort_by_row(hl_wide* w, const int32_t* table_of_entry, const int32_t* d_n, int64_t n_max, int32_t** out_vals,
                    cudaStream_t stream) {
    int32_t *k1, *v1;
    int32_t st = radix_sort_pairs(w->sort_keys, w->sort_vals, d_n, n_max, 31, w->sort_hist, w->status, &k1, &v1, stream);
    if (st != HL_OK) return st;
    // the result sits in buffer `cur`; the second sort starts from buffer 0, so bring it there if needed
    const int cur = v1 == w->sort_vals[0] ? 0 : 1;
    if (cur == 1) {
        HL_CUDA_TRY(cudaMemcpyAsync(w->sort_vals[0], w->sort_vals[1], sizeof(int32_t) * n_max, cudaMemcpyDeviceToDevice,
                                    stream));
    }
    k_wide_gather_key<<<grid_for(n_max, kThreads, 8 * w->sms), kThreads, 0, stream>>>(w->sort_vals[0], table_of_entry,
                                                                                      d_n, n_max, w->sort_keys[0]);
    note_launches(1);
    HL_LAUNCH_CHECK();
    int32_t* k2;
    return radix_sort_pairs(w->sort_keys, w->sort_vals, d_n, n_max, bits_for(w->T - 1), w->sort_hist, w->status, &k2,
                            out_vals, stream);
}

// cold lookups of X as (table, index, position): a lookup whose row is popular gets its slot at once
__global__ void __launch_bounds__(kThreads) k_wide_classify(const long long* __restrict__ rows,
                                                            const int32_t* __restrict__ offsets,
                                                            const int32_t* __restrict__ d_n_non, int max_batch,
                                                            int bags_per_sample_all, int64_t cap, int64_t N,
                                                            HashProbe probe, const int64_t* __restrict__ table_base,
                                                            int T, int32_t* __restrict__ slots, int32_t* c_tab,
                                                            int32_t* c_idx, int32_t* c_pos, int32_t* sort_key,
                                                            int32_t* sort_val, int32_t* d_n_cold_lookups,
                                                            int64_t max_nnz, int32_t* status) {
    int n_non = *d_n_non;
    n_non = n_non < 0 ? 0 : (n_non > max_batch ? max_batch : n_non);
    int64_t L = offsets[(int64_t)n_non * bags_per_sample_all];
    if (L > cap) L = cap;
    for (int64_t j = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; j < L; j += (int64_t)gridDim.x * blockDim.x) {
        const long long g = rows[j];
        if (g < 0 || g >= N) {
            if (g >= N) set_status(status, HL_EBOUNDS);
            slots[j] = -1;
            continue;
        }
        const int32_t s = probe.slot(g);
        if (s >= 0) {
            slots[j] = s;
            continue;
        }
        int lo = 0, hi = T;
        while (hi - lo > 1) {
            const int mid = (lo + hi) >> 1;
            if (table_base[mid] <= g) lo = mid;
            else hi = mid;
        }
        const int32_t i = atomicAdd(d_n_cold_lookups, 1);
        if (i >= max_nnz) continue;
        c_tab[i] = lo;
        c_idx[i] = (int32_t)(g - table_base[lo]);
        c_pos[i] = (int32_t)j;
        sort_key[i] = c_idx[i];
        sort_val[i] = i;
    }
}

// head[j] = 1 where the j-th cold lookup in row order addresses another row than the one before
__global__ void __launch_bounds__(kThreads) k_wide_heads(const int32_t* __restrict__ ent,
                                                         const int32_t* __restrict__ c_tab,
                                                         const int32_t* __restrict__ c_idx, const int32_t* d_n,
                                                         int64_t n_max, int32_t* __restrict__ heads) {
    int64_t n = *d_n;
    n = n < n_max ? n : n_max;
    for (int64_t j = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; j < n; j += (int64_t)gridDim.x * blockDim.x) {
        const int32_t e = ent[j], p = j > 0 ? ent[j - 1] : -1;
        heads[j] = (j == 0 || c_tab[e] != c_tab[p] || c_idx[e] != c_idx[p]) ? 1 : 0;
    }
}

__global__ void __launch_bounds__(kThreads) k_wide_assign(const int32_t* __restrict__ ent,
                                                          const int32_t* __restrict__ c_tab,
                                                          const int32_t* __restrict__ c_idx,
                                                          const int32_t* __restrict__ c_pos, const int32_t* d_n,
                                                          int64_t n_max, const int32_t* __restrict__ rank_excl,
                                                          const int64_t* __restrict__ table_base, int64_t slot0,
                                                          int64_t staging_cap, int64_t cap_ids,
                                                          int32_t* __restrict__ slots, long long* __restrict__ cold_rows,
                                                          int64_t* __restrict__ d_n_cold, int32_t* status) {
    int64_t n = *d_n;
    n = n < n_max ? n : n_max;
    if (blockIdx.x == 0 && threadIdx.x == 0) {
        int64_t distinct = n > 0 ? rank_excl[n] : 0;
        if (distinct > staging_cap) {
            set_status(status, HL_ECAPACITY);
            distinct = staging_cap;
        }
        *d_n_cold = distinct;
    }
    for (int64_t j = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; j < n; j += (int64_t)gridDim.x * blockDim.x) {
        const int32_t e = ent[j], p = j > 0 ? ent[j - 1] : -1;
        const bool head = j == 0 || c_tab[e] != c_tab[p] || c_idx[e] != c_idx[p];
        const int64_t rank = head ? rank_excl[j] : rank_excl[j] - 1;
        const int64_t where = c_pos[e];
        if (where < 0 || where >= cap_ids || rank < 0) continue;
        if (rank < staging_cap) {
            if (head) cold_rows[rank] = table_base[c_tab[e]] + c_idx[e];
            slots[where] = (int32_t)(slot0 + rank);
        } else {
            slots[where] = -1;      // no room to stage this row: the lookup is dropped, the status word says so
        }
    }
}

}  // namespace
}  // namespace hl

extern "C" int32_t hl_wide_profile_hot(hl_wide* w, const hl_batch* b, int32_t reset, int32_t finalize, int32_t policy,
                                       int64_t p_num, int64_t p_den, int32_t row_bytes, int64_t* d_hot_rows,
                                       int64_t* d_n_hot, void* stream_) {
    if (!w) return HL_EINVAL;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    const int64_t E = w->counter_slots;
    if (reset) {
        HL_CUDA_TRY(cudaMemsetAsync(w->c_keys, 0xff, sizeof(long long) * E, stream));
        HL_CUDA_TRY(cudaMemsetAsync(w->c_cnt, 0, sizeof(uint32_t) * E, stream));
        HL_CUDA_TRY(cudaMemsetAsync(w->sel, 0, sizeof(SelectState), stream));
    }
    if (b) {
        if (b->batch < 1 || b->batch > w->max_batch || b->nnz < 0 || b->nnz > w->max_nnz || !b->offsets ||
            (b->nnz > 0 && !b->indices))
            return HL_EINVAL;
        const int64_t bags_per_table = (int64_t)b->batch * w->S;
        const int64_t n_bags = bags_per_table * w->T;
        k_wide_count<<<grid_for(n_bags, kThreads, w->sms * 8), kThreads, 0, stream>>>(
            b->indices, b->offsets, n_bags, bags_per_table, w->table_base, w->c_keys, w->c_cnt, (uint64_t)(E - 1),
            w->sel, w->status);
        note_launches(1);
        HL_LAUNCH_CHECK();
    }
    if (!finalize) return HL_OK;
    if (!d_hot_rows || !d_n_hot) return HL_EINVAL;
    long long k = 0, share_num = 0, share_den = 1;
    switch (policy) {
        case HL_HOT_TOPK_ROWS: k = p_num; break;
        case HL_HOT_BUDGET_BYTES:
            if (row_bytes < 1) return HL_EINVAL;
            k = p_num / row_bytes;
            break;
        case HL_HOT_FRACTION_ROWS:
            if (p_den <= 0 || p_num < 0) return HL_EINVAL;
            k = (long long)(((__int128)w->N * p_num) / p_den);
            break;
        case HL_HOT_MIN_SHARE:
            if (p_den <= 0 || p_num <= 0) return HL_EINVAL;
            k = w->hot_cap;
            share_num = p_num;
            share_den = p_den;
            break;
        default: return HL_EINVAL;
    }
    if (k < 0) return HL_EINVAL;
    if (k > w->hot_cap) k = w->hot_cap;
    // the counted rows in ascending order of their global id, with their counts: then the selection is the one of the
    // dense counter, over positions instead of rows (ties at the threshold go to the smaller position = smaller id)
    HL_CUDA_TRY(cudaMemsetAsync(w->n_seen, 0, 4 * sizeof(int32_t), stream));
    k_wide_entries<<<grid_for(E, kThreads, w->sms * 8), kThreads, 0, stream>>>(
        w->c_keys, w->c_cnt, E, w->table_base, w->T, w->n_seen, w->e_tab, w->e_idx, w->e_cnt, w->sort_keys[0],
        w->sort_vals[0]);
    note_launches(1);
    HL_LAUNCH_CHECK();
    int32_t* order;
    int32_t st = sort_by_row(w, w->e_tab, w->n_seen, E, &order, stream);
    if (st != HL_OK) return st;
    k_wide_row_order<<<grid_for(E, kThreads, w->sms * 8), kThreads, 0, stream>>>(order, w->e_cnt, w->n_seen, E, w->s_cnt,
                                                                               w->s_ent);
    note_launches(1);
    HL_LAUNCH_CHECK();
    st = select_rows_by_count(w->s_cnt, E, w->sel, w->sel_gt, w->sel_eq, k, share_num, share_den, w->hot_cap,
                              w->sel_idx, d_n_hot, w->status, w->sms, stream);
    if (st != HL_OK) return st;
    k_wide_hot_rows<<<grid_for(w->hot_cap, kThreads, w->sms * 8), kThreads, 0, stream>>>(
        w->sel_idx, d_n_hot, w->hot_cap, w->s_ent, w->e_tab, w->e_idx, w->table_base,
        reinterpret_cast<long long*>(d_hot_rows));
    note_launches(1);
    HL_LAUNCH_CHECK();
    return HL_OK;
}

extern "C" int32_t hl_wide_build_remap(hl_wide* w, const int64_t* d_hot_rows, const int64_t* d_n_hot, void* stream_) {
    if (!w || !d_hot_rows || !d_n_hot) return HL_EINVAL;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    HL_CUDA_TRY(cudaMemsetAsync(w->r_keys, 0xff, sizeof(long long) * w->remap_slots, stream));
    if (w->hot_cap > 0) {
        k_wide_remap<<<grid_for(w->hot_cap, kThreads, w->sms * 8), kThreads, 0, stream>>>(
            reinterpret_cast<const long long*>(d_hot_rows), d_n_hot, w->hot_cap, w->N, w->r_keys, w->r_vals,
            (uint64_t)(w->remap_slots - 1), w->status);
        note_launches(1);
        HL_LAUNCH_CHECK();
    }
    return HL_OK;
}

extern "C" int32_t hl_wide_index_cold(hl_wide* w, const int32_t* d_non_offsets, const int64_t* d_non_rows,
                                      int64_t non_cap, const int32_t* d_n_non, int32_t* d_non_slots,
                                      int64_t* d_cold_rows, int64_t* d_n_cold, void* stream_) {
    if (!w || !d_non_offsets || !d_n_non || !d_cold_rows || !d_n_cold) return HL_EINVAL;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    if (w->max_nnz == 0) {
        HL_CUDA_TRY(cudaMemsetAsync(d_n_cold, 0, sizeof(int64_t), stream));
        return HL_OK;
    }
    if (!d_non_rows || !d_non_slots) return HL_EINVAL;
    HL_CUDA_TRY(cudaMemsetAsync(w->cold_n, 0, 4 * sizeof(int32_t), stream));
    const HashProbe probe{w->r_keys, w->r_vals, (uint64_t)(w->remap_slots - 1)};
    const int grid = grid_for(w->max_nnz, kThreads, 8 * w->sms);
    k_wide_classify<<<grid, kThreads, 0, stream>>>(reinterpret_cast<const long long*>(d_non_rows), d_non_offsets, d_n_non,
                                                   w->max_batch, w->T * w->S, non_cap, w->N, probe, w->table_base, w->T,
                                                   d_non_slots, w->cold_tab, w->cold_idx, w->cold_pos, w->sort_keys[0],
                                                   w->sort_vals[0], w->cold_n, w->max_nnz, w->status);
    note_launches(1);
    HL_LAUNCH_CHECK();
    int32_t* order;
    int32_t st = sort_by_row(w, w->cold_tab, w->cold_n, w->max_nnz, &order, stream);
    if (st != HL_OK) return st;
    k_wide_heads<<<grid, kThreads, 0, stream>>>(order, w->cold_tab, w->cold_idx, w->cold_n, w->max_nnz, w->cold_rank);
    note_launches(1);
    HL_LAUNCH_CHECK();
    st = exclusive_scan_i32(w->cold_rank, w->cold_rank, w->cold_n, w->max_nnz, w->cold_tiles, w->status, stream);
    if (st != HL_OK) return st;
    k_wide_assign<<<grid, kThreads, 0, stream>>>(order, w->cold_tab, w->cold_idx, w->cold_pos, w->cold_n, w->max_nnz,
                                                 w->cold_rank, w->table_base, w->hot_cap, w->staging_cap, non_cap,
                                                 d_non_slots, reinterpret_cast<long long*>(d_cold_rows), d_n_cold,
                                                 w->status);
    note_launches(1);
    HL_LAUNCH_CHECK();
    return HL_OK;
}
