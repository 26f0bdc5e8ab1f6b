// Context, workspace carving and status of the Hotline library.
#include <stdlib.h>
#include <string.h>

#include "hl_common.cuh"

namespace hl {
namespace {

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

bool geometry_ok(const hl_geometry* g, int64_t* total_rows) {
    if (!g || g->num_tables < 1 || g->dim < 4 || (g->dim & 3) || g->bags_per_sample < 1 || !g->table_rows)
        return false;
    int64_t n = 0;
    for (int t = 0; t < g->num_tables; ++t) {
        if (g->table_rows[t] < 1) return false;
        n += g->table_rows[t];
        if (n >= (int64_t(1) << 31)) return false;   // global row ids are int32
    }
    *total_rows = n;
    return true;
}

int64_t hist_words(int64_t max_nnz) { return sort_hist_words(max_nnz); }

// Lays the regions out over `base` (nullptr: size only).  Returns the bytes used.
size_t carve(char* base, const hl_geometry* g, int64_t N, int32_t max_batch, int64_t max_nnz, int64_t hot_cap,
             int64_t staging_cap, Regions* r, int64_t* n_remap_blocks, int64_t* n_sel_tiles) {
    Carver c{base};
    const int64_t T = g->num_tables, S = g->bags_per_sample, D = g->dim;
    const int64_t max_bags = T * (int64_t)max_batch * S;
    const int64_t nnz = max_nnz > 0 ? max_nnz : 1;
    *n_remap_blocks = div_up(N, kRemapRowsPerBlock) + 1;
    *n_sel_tiles = div_up(N, kSelTile);
    r->status = c.take<int32_t>(8);
    r->table_base = c.take<int64_t>(T + 1);
    r->table_ptrs = c.take<unsigned char*>(T);
    r->remap = c.take<RemapBlock>(*n_remap_blocks);
    r->counts = c.take<uint32_t>(N);
    r->sel = c.take<SelectState>(1);
    r->sel_gt = c.take<uint32_t>(*n_sel_tiles + 2);
    r->sel_eq = c.take<uint32_t>(*n_sel_tiles + 2);
    r->frag_flags = c.take<uint8_t>(max_batch);
    r->frag_scan = c.take<int32_t>(max_bags + 2);
    r->frag_tiles = c.take<int32_t>(scan_tile_words(max_bags));
    for (int i = 0; i < 2; ++i) {
        r->bwd_keys[i] = c.take<int32_t>(nnz);
        r->bwd_vals[i] = c.take<int32_t>(nnz);
    }
    r->bwd_hist = c.take<uint32_t>(hist_words(nnz));
    r->bwd_part = c.take<float>(2 * div_up(nnz, kBwdChunk) * D + bwd_span_list_words(nnz));
    r->bwd_n = c.take<int32_t>(4);
    for (int i = 0; i < 2; ++i) {
        r->cold_keys[i] = c.take<int32_t>(nnz);
        r->cold_vals[i] = c.take<int32_t>(nnz);
    }
    r->cold_hist = c.take<uint32_t>(hist_words(nnz));
    r->cold_rank = c.take<int32_t>(nnz + 2);
    r->cold_tiles = c.take<int32_t>(scan_tile_words(nnz));
    r->cold_n = c.take<int32_t>(4);
    (void)hot_cap;
    (void)staging_cap;
    return (c.off + 255) & ~size_t(255);
}

}  // namespace
}  // namespace hl

using namespace hl;

extern "C" size_t hl_workspace_bytes(const hl_geometry* geom, int32_t max_batch, int64_t max_nnz,
                                     int64_t hot_cap_rows, int64_t staging_cap_rows) {
    int64_t N;
    if (!geometry_ok(geom, &N) || max_batch < 1 || max_nnz < 0 || hot_cap_rows < 0 || staging_cap_rows < 0) return 0;
    Regions r;
    int64_t a, b;
    return carve(nullptr, geom, N, max_batch, max_nnz, hot_cap_rows, staging_cap_rows, &r, &a, &b);
}

extern "C" int32_t hl_create(hl_ctx** out, const hl_geometry* geom, int32_t max_batch, int64_t max_nnz,
                             int64_t hot_cap_rows, int64_t staging_cap_rows, void* d_workspace, size_t ws_bytes) {
    if (!out) return HL_EINVAL;
    *out = nullptr;
    int64_t N;
    if (!geometry_ok(geom, &N) || max_batch < 1 || max_nnz < 0 || hot_cap_rows < 0 || staging_cap_rows < 0)
        return HL_EINVAL;
    const int64_t max_bags = (int64_t)geom->num_tables * max_batch * geom->bags_per_sample;
    if (max_bags >= (int64_t(1) << 30) || max_nnz >= (int64_t(1) << 30)) return HL_EINVAL;   // 30-bit chain values
    if (hot_cap_rows + staging_cap_rows >= (int64_t(1) << 31) - 2) return HL_EINVAL;
    if (!d_workspace || (reinterpret_cast<uintptr_t>(d_workspace) & 255)) return HL_EINVAL;

    hl_ctx* ctx = static_cast<hl_ctx*>(calloc(1, sizeof(hl_ctx)));
    if (!ctx) return HL_EINVAL;
    ctx->T = geom->num_tables;
    ctx->D = geom->dim;
    ctx->S = geom->bags_per_sample;
    ctx->N = N;
    ctx->max_batch = max_batch;
    ctx->max_nnz = max_nnz;
    ctx->max_bags = max_bags;
    ctx->hot_cap = hot_cap_rows;
    ctx->staging_cap = staging_cap_rows;
    const size_t need = carve(static_cast<char*>(d_workspace), geom, N, max_batch, max_nnz, hot_cap_rows,
                              staging_cap_rows, &ctx->r, &ctx->n_remap_blocks, &ctx->n_sel_tiles);
    if (need > ws_bytes) {
        free(ctx);
        return HL_ECAPACITY;
    }
    if (cudaGetDevice(&ctx->device) != cudaSuccess ||
        cudaDeviceGetAttribute(&ctx->sms, cudaDevAttrMultiProcessorCount, ctx->device) != cudaSuccess) {
        free(ctx);
        return HL_ECUDA;
    }
    ctx->mover_ctas = kReadCtasDefault;
    ctx->scatter_ctas = kMoverCtasDefault;
    ctx->test_poll_limit = 0;
    ctx->test_stall_tile = -1;
    ctx->h_table_base = static_cast<int64_t*>(malloc(sizeof(int64_t) * (ctx->T + 1)));
    if (!ctx->h_table_base) {
        free(ctx);
        return HL_EINVAL;
    }
    ctx->h_table_base[0] = 0;
    for (int t = 0; t < ctx->T; ++t) ctx->h_table_base[t + 1] = ctx->h_table_base[t] + geom->table_rows[t];

    cudaError_t e = cudaMemcpy(ctx->r.table_base, ctx->h_table_base, sizeof(int64_t) * (ctx->T + 1),
                               cudaMemcpyHostToDevice);
    if (e == cudaSuccess) e = cudaMemset(ctx->r.status, 0, 8 * sizeof(int32_t));
    if (e == cudaSuccess) e = cudaMemset(ctx->r.remap, 0, sizeof(RemapBlock) * ctx->n_remap_blocks);
    if (e == cudaSuccess) e = cudaMemset(ctx->r.counts, 0, sizeof(uint32_t) * N);
    if (e == cudaSuccess) e = cudaMemset(ctx->r.sel, 0, sizeof(SelectState));
    if (e == cudaSuccess) e = cudaMemset(ctx->r.frag_tiles, 0, sizeof(int32_t) * scan_tile_words(max_bags));
    if (e == cudaSuccess) e = cudaMemset(span_count_of(ctx), 0, 8 * sizeof(int32_t));   // kept zero between backward calls
    if (e == cudaSuccess) e = cudaDeviceSynchronize();
    if (e != cudaSuccess) {
        free(ctx->h_table_base);
        free(ctx);
        return HL_ECUDA;
    }
    *out = ctx;
    return HL_OK;
}

extern "C" int32_t hl_set_host_tables(hl_ctx* ctx, float* const* h_table_bases) {
    if (!ctx) return HL_EINVAL;
    if (!h_table_bases) {
        ctx->per_table = 0;
        return HL_OK;
    }
    for (int t = 0; t < ctx->T; ++t)
        if (!h_table_bases[t] || (reinterpret_cast<uintptr_t>(h_table_bases[t]) & 15)) return HL_EINVAL;
    HL_CUDA_TRY(cudaDeviceSynchronize());      // no kernel may still be reading the previous addresses
    HL_CUDA_TRY(cudaMemcpy(ctx->r.table_ptrs, h_table_bases, sizeof(float*) * ctx->T, cudaMemcpyHostToDevice));
    ctx->per_table = 1;
    return HL_OK;
}

extern "C" int32_t hl_set_mover_ctas(hl_ctx* ctx, int32_t read_ctas, int32_t write_ctas) {
    if (!ctx || read_ctas < 0 || write_ctas < 0) return HL_EINVAL;
    const int most = 2 * ctx_sms(ctx);
    ctx->mover_ctas = read_ctas == 0 ? kReadCtasDefault : (read_ctas < most ? read_ctas : most);
    ctx->scatter_ctas = write_ctas == 0 ? kMoverCtasDefault : (write_ctas < most ? write_ctas : most);
    return HL_OK;
}

extern "C" int32_t hl_set_kernel_width(hl_ctx* ctx, int32_t fwd_ctas_per_sm, int32_t bwd_ctas_per_sm) {
    if (!ctx || fwd_ctas_per_sm < 0 || bwd_ctas_per_sm < 0 || fwd_ctas_per_sm > 32 || bwd_ctas_per_sm > 32)
        return HL_EINVAL;
    ctx->fwd_ctas = fwd_ctas_per_sm;
    ctx->bwd_ctas = bwd_ctas_per_sm;
    return HL_OK;
}

extern "C" int32_t hl_test_bounded_waits(hl_ctx* ctx, int32_t poll_limit, int64_t stall_tile) {
    if (!ctx || poll_limit < 0) return HL_EINVAL;
    ctx->test_poll_limit = poll_limit;
    ctx->test_stall_tile = poll_limit > 0 ? stall_tile : -1;
    return HL_OK;
}

extern "C" int32_t hl_timing_enable(hl_ctx* ctx, int32_t on) {
    if (!ctx) return HL_EINVAL;
    if (on && !ctx->timer[0][0]) {
        for (int w = 0; w < HL_TIMER_COUNT; ++w)
            for (int e = 0; e < 2; ++e) HL_CUDA_TRY(cudaEventCreate(&ctx->timer[w][e]));
    }
    ctx->timing_on = on ? 1 : 0;
    return HL_OK;
}

extern "C" int32_t hl_timing_read(hl_ctx* ctx, int32_t which, float* ms) {
    if (!ctx || !ms || which < 0 || which >= HL_TIMER_COUNT || !ctx->timer[which][0]) return HL_EINVAL;
    if (cudaEventElapsedTime(ms, ctx->timer[which][0], ctx->timer[which][1]) != cudaSuccess) {
        cudaGetLastError();
        return HL_EINVAL;   // never recorded, or not finished yet
    }
    return HL_OK;
}

extern "C" int32_t hl_destroy(hl_ctx* ctx) {
    if (!ctx) return HL_EINVAL;
    for (int w = 0; w < HL_TIMER_COUNT; ++w)
        for (int e = 0; e < 2; ++e)
            if (ctx->timer[w][e]) cudaEventDestroy(ctx->timer[w][e]);
    free(ctx->h_table_base);
    free(ctx);
    return HL_OK;
}

extern "C" int32_t hl_status(hl_ctx* ctx) {
    if (!ctx) return HL_EINVAL;
    HL_CUDA_TRY(cudaDeviceSynchronize());
    int32_t st = 0;
    HL_CUDA_TRY(cudaMemcpy(&st, ctx->r.status, sizeof(int32_t), cudaMemcpyDeviceToHost));
    if (st != 0) HL_CUDA_TRY(cudaMemset(ctx->r.status, 0, sizeof(int32_t)));
    return st;
}

namespace hl {
unsigned long long launches_so_far();
}

extern "C" uint64_t hl_launch_count(void) { return hl::launches_so_far(); }

// Host-resident memory that the current device reads and writes in place.  It is unified memory whose preferred
// location is the CPU and which the device is advised to map ("accessed by"): the pages stay in host DRAM, nothing
// migrates, and -- unlike memory from cudaHostAlloc / cudaHostRegister, which the device maps in 4 KB pages -- the
// device maps it in large pages.  That matters for a table of tens of GB read at random: with 4 KB mappings
// every fresh row paid an address-translation miss (measured 20-24 ns per 256-byte row, 10-13 GB/s); with this
// allocation the same rows move at 46 GB/s.
extern "C" void* hl_host_alloc(size_t bytes) {
    void* p = nullptr;
    int dev = 0;
    if (bytes == 0 || cudaGetDevice(&dev) != cudaSuccess) return nullptr;
    if (cudaMallocManaged(&p, bytes, cudaMemAttachGlobal) == cudaSuccess) {
        if (cudaMemAdvise(p, bytes, cudaMemAdviseSetPreferredLocation, cudaCpuDeviceId) == cudaSuccess &&
            cudaMemAdvise(p, bytes, cudaMemAdviseSetAccessedBy, dev) == cudaSuccess &&
            cudaMemPrefetchAsync(p, bytes, cudaCpuDeviceId, 0) == cudaSuccess &&   // populate the pages in host DRAM
            cudaDeviceSynchronize() == cudaSuccess)
            return p;
        cudaGetLastError();
        cudaFree(p);
    }
    cudaGetLastError();
    // Unified memory refused the size (on the bench platform one allocation stops between 66 and 70 GB): plain
    // pinned, mapped host memory still works as a table, with 4 KB device mappings.
    p = nullptr;
    if (cudaHostAlloc(&p, bytes, cudaHostAllocMapped | cudaHostAllocPortable) != cudaSuccess) {
        cudaGetLastError();
        return nullptr;
    }
    return p;
}

extern "C" int32_t hl_host_free(void* p) {
    if (!p) return HL_OK;
    cudaPointerAttributes attr;
    if (cudaPointerGetAttributes(&attr, p) != cudaSuccess) {
        cudaGetLastError();
        return HL_ECUDA;
    }
    if (attr.type == cudaMemoryTypeManaged) HL_CUDA_TRY(cudaFree(p));
    else HL_CUDA_TRY(cudaFreeHost(p));
    return HL_OK;
}

extern "C" const char* hl_strerror(int32_t status) {
    switch (status) {
        case HL_OK: return "ok";
        case HL_EINVAL: return "invalid argument or malformed data";
        case HL_EBOUNDS: return "index outside its table or slot outside the cache";
        case HL_ECAPACITY: return "output buffer, hot cache or staging area too small";
        case HL_ECUDA: return "CUDA runtime error";
        case HL_ETIMEOUT: return "device-side wait timed out";
        default: return "unknown status";
    }
}
