// The software-pipelined schedule over mini-batches, issued from native code: the same order of calls, streams and
// events as the Python scheduler, without an interpreter between the launches (a mini-batch is about 32 kernels, 10
// memsets and 25 event operations; issued from Python that alone takes 0.2 ms).
//
//   stream A     hl_fragment(j+L)
//   stream C     hl_index_cold(j+L)            after A;  needs the cold rows of j+L-1 (same stream, in order)
//   stream B     hl_embbag_bwd_prepare2(j+L)   after C
//   link stream  hl_forward_cold(j)            after the backward of j-1;  then
//                hl_stage_cold(j+1)            after the write-back of j-1 (host rows final, window free)
//   main stream  forward O, update O, [rows of j staged and forwarded] forward X, update X          mini-batch j
//   write-back   hl_scatter_cold_at(j)         after the update of X
//
// L = n_sets - 2 mini-batches of index-only work ahead; set j % n_sets holds mini-batch j; window j % 2 its cold rows.
#include "hl_common.cuh"

#include <new>
#include <vector>

struct hl_pipe {
    hl_ctx* ctx;
    float* cache;
    float* host_table;
    int64_t window_rows;
    int n_sets, n_dense;
    std::vector<hl_pipe_set> sets;
    cudaStream_t main, sa, sb, sc, link, wb;
    struct Events {
        cudaEvent_t inputs, frag, index, prep, gather, forward, x, scatter;
    };
    std::vector<Events> ev;
    int64_t j_indexed, j_submitted, j_done;
    cudaEvent_t time_fwd[4];     // one-shot: recorded around the two forward calls of the next step
};

namespace {

#define HL_PIPE_TRY(expr)                         \
    do {                                          \
        const int32_t st__ = (expr);              \
        if (st__ != HL_OK) return st__;           \
    } while (0)

int32_t wait(cudaStream_t s, cudaEvent_t e) { return cudaStreamWaitEvent(s, e, 0) == cudaSuccess ? HL_OK : HL_ECUDA; }
int32_t record(cudaEvent_t e, cudaStream_t s) { return cudaEventRecord(e, s) == cudaSuccess ? HL_OK : HL_ECUDA; }

// fragment, cold-row search and backward sort of the next mini-batch (index-only: nothing here touches a row)
int32_t submit_index(hl_pipe* p, const hl_batch* b, const float* d_dense) {
    const int64_t j = p->j_indexed;
    const int n = p->n_sets;
    hl_pipe_set& st = p->sets[j % n];
    hl_pipe::Events& e = p->ev[j % n];
    hl_pipe_set* prev = j >= 1 ? &p->sets[(j - 1) % n] : nullptr;
    const int64_t w = (j % 2) * p->window_rows;
    HL_PIPE_TRY(wait(p->sa, e.inputs));
    if (j >= n) HL_PIPE_TRY(wait(p->sa, e.scatter));      // the buffers of this set were mini-batch j-n_sets's
    HL_PIPE_TRY(hl_fragment(p->ctx, b, d_dense, d_dense ? p->n_dense : 0, st.perm, st.counts, &st.pop, &st.non,
                            d_dense ? st.dense_out : nullptr, p->sa));
    HL_PIPE_TRY(record(e.frag, p->sa));
    HL_PIPE_TRY(wait(p->sc, e.frag));
    if (j >= n) HL_PIPE_TRY(wait(p->sc, e.scatter));
    HL_PIPE_TRY(hl_index_cold(p->ctx, &st.non, st.counts + 1, w, p->window_rows, st.cold_rows, st.n_cold,
                              prev ? prev->cold_rows : nullptr, prev ? prev->n_cold : nullptr, st.fwd_src, p->sc));
    HL_PIPE_TRY(record(e.index, p->sc));
    HL_PIPE_TRY(wait(p->sb, e.index));
    HL_PIPE_TRY(hl_embbag_bwd_prepare2(p->ctx, &st.pop, st.counts, &st.non, st.counts + 1, st.sorted_slots,
                                       st.sorted_bags, st.sorted_n, p->sb));
    HL_PIPE_TRY(record(e.prep, p->sb));
    p->j_indexed += 1;
    return HL_OK;
}

// the host read of the oldest indexed mini-batch whose rows are not staged yet
int32_t submit_link(hl_pipe* p) {
    const int64_t j = p->j_submitted;
    const int n = p->n_sets;
    hl_pipe_set& st = p->sets[j % n];
    const int64_t w = (j % 2) * p->window_rows;
    HL_PIPE_TRY(wait(p->link, p->ev[j % n].index));
    if (j >= 2) HL_PIPE_TRY(wait(p->link, p->ev[(j - 2) % n].scatter));   // host rows of j-2 final, its window free
    if (j >= 1) HL_PIPE_TRY(wait(p->link, p->ev[(j - 1) % n].forward));   // j-1 took what it needs out of the window
    HL_PIPE_TRY(hl_stage_cold(p->ctx, p->host_table, p->cache, w, p->window_rows, st.cold_rows, st.n_cold,
                              j >= 1 ? st.fwd_src : nullptr, p->link));
    HL_PIPE_TRY(record(p->ev[j % n].gather, p->link));
    p->j_submitted += 1;
    return HL_OK;
}

}  // namespace

extern "C" hl_pipe* hl_pipe_create(hl_ctx* ctx, float* d_cache, float* host_table, int64_t window_rows,
                                   int32_t n_sets, const hl_pipe_set* sets, int32_t n_dense, void* main_stream) {
    if (!ctx || !d_cache || !host_table || !sets || n_sets < 3 || n_sets > 16 || window_rows < 0 ||
        2 * window_rows > ctx->staging_cap || n_dense < 0)
        return nullptr;
    for (int i = 0; i < n_sets; ++i) {
        const hl_pipe_set& s = sets[i];
        if (!s.perm || !s.counts || !s.pop.offsets || !s.non.offsets || !s.cold_rows || !s.n_cold || !s.fwd_src ||
            !s.pooled_pop || !s.pooled_non || !s.sorted_n || (n_dense > 0 && !s.dense_out))
            return nullptr;
        if (ctx->max_nnz > 0 && (!s.pop.ids || !s.non.ids || !s.sorted_slots || !s.sorted_bags)) return nullptr;
    }
    hl_pipe* p = new (std::nothrow) hl_pipe();
    if (!p) return nullptr;
    p->ctx = ctx;
    p->cache = d_cache;
    p->host_table = host_table;
    p->window_rows = window_rows;
    p->n_sets = n_sets;
    p->n_dense = n_dense;
    p->sets.assign(sets, sets + n_sets);
    p->main = static_cast<cudaStream_t>(main_stream);
    p->j_indexed = p->j_submitted = p->j_done = 0;
    for (auto& t : p->time_fwd) t = nullptr;
    int lo = 0, hi = 0;
    cudaDeviceGetStreamPriorityRange(&lo, &hi);          // hi = numerically lowest = highest priority
    cudaStream_t* side[5] = {&p->sa, &p->sb, &p->sc, &p->link, &p->wb};
    bool ok = true;
    for (auto s : side) {
        *s = nullptr;
        ok = ok && cudaStreamCreateWithPriority(s, cudaStreamNonBlocking, hi) == cudaSuccess;
    }
    p->ev.resize(n_sets);
    for (auto& e : p->ev) {
        cudaEvent_t* all[8] = {&e.inputs, &e.frag, &e.index, &e.prep, &e.gather, &e.forward, &e.x, &e.scatter};
        for (auto x : all) {
            *x = nullptr;
            ok = ok && cudaEventCreateWithFlags(x, cudaEventDisableTiming) == cudaSuccess;
        }
    }
    if (!ok) {
        hl_pipe_destroy(p);
        return nullptr;
    }
    return p;
}

extern "C" void hl_pipe_destroy(hl_pipe* p) {
    if (!p) return;
    cudaStream_t side[5] = {p->sa, p->sb, p->sc, p->link, p->wb};
    for (auto s : side)
        if (s) {
            cudaStreamSynchronize(s);
            cudaStreamDestroy(s);
        }
    for (auto& e : p->ev) {
        cudaEvent_t all[8] = {e.inputs, e.frag, e.index, e.prep, e.gather, e.forward, e.x, e.scatter};
        for (auto x : all)
            if (x) cudaEventDestroy(x);
    }
    delete p;
}

extern "C" int32_t hl_pipe_submit(hl_pipe* p, const hl_batch* b, const float* d_dense) {
    if (!p || !b) return HL_EINVAL;
    if (p->j_indexed - p->j_done >= p->n_sets - 1) return HL_ECAPACITY;    // every spare buffer set is in flight
    HL_PIPE_TRY(record(p->ev[p->j_indexed % p->n_sets].inputs, p->main));   // the inputs are ready at this point
    HL_PIPE_TRY(submit_index(p, b, d_dense));
    if (p->j_submitted == p->j_done) HL_PIPE_TRY(submit_link(p));           // nothing staged ahead yet
    return HL_OK;
}

extern "C" int32_t hl_pipe_step(hl_pipe* p, const float* d_grad_pop, const float* d_grad_non, float lr,
                                const hl_batch* next, const float* d_next_dense, int32_t* set_index) {
    if (!p || !d_grad_pop || !d_grad_non) return HL_EINVAL;
    const int64_t j = p->j_done;
    if (p->j_submitted < j + 1) return HL_EINVAL;          // hl_pipe_submit first
    const int n = p->n_sets;
    hl_pipe_set& st = p->sets[j % n];
    hl_pipe::Events& e = p->ev[j % n];
    const int64_t w0 = (j % 2) * p->window_rows, w1 = ((j + 1) % 2) * p->window_rows;
    if (next) {
        if (p->j_indexed - j >= n - 1) return HL_ECAPACITY;
        HL_PIPE_TRY(record(p->ev[p->j_indexed % n].inputs, p->main));
    }
    HL_PIPE_TRY(wait(p->main, e.index));
    if (j >= 1) {
        // rows shared with mini-batch j-1 come out of its staging window once its backward is done
        HL_PIPE_TRY(wait(p->link, e.index));
        HL_PIPE_TRY(wait(p->link, p->ev[(j - 1) % n].x));
        HL_PIPE_TRY(hl_forward_cold(p->ctx, p->cache, w1, w0, p->window_rows, st.fwd_src, st.n_cold, p->link));
    }
    HL_PIPE_TRY(record(e.forward, p->link));
    if (p->j_submitted < p->j_indexed) HL_PIPE_TRY(submit_link(p));         // mini-batch j+1, indexed earlier
    if (next) {
        HL_PIPE_TRY(submit_index(p, next, d_next_dense));
        if (p->j_submitted == j + 1) HL_PIPE_TRY(submit_link(p));           // j+1 was indexed only just now
    }
    if (p->time_fwd[0]) HL_PIPE_TRY(record(p->time_fwd[0], p->main));
    HL_PIPE_TRY(hl_embbag_fwd(p->ctx, p->cache, &st.pop, st.counts, st.pooled_pop, p->main));
    if (p->time_fwd[1]) HL_PIPE_TRY(record(p->time_fwd[1], p->main));
    HL_PIPE_TRY(wait(p->main, e.prep));
    HL_PIPE_TRY(hl_embbag_bwd_apply2(p->ctx, p->cache, st.sorted_slots, st.sorted_bags, st.sorted_n, 0, d_grad_pop, lr,
                                     p->main));
    HL_PIPE_TRY(wait(p->main, e.gather));
    HL_PIPE_TRY(wait(p->main, e.forward));
    if (p->time_fwd[2]) HL_PIPE_TRY(record(p->time_fwd[2], p->main));
    HL_PIPE_TRY(hl_embbag_fwd(p->ctx, p->cache, &st.non, st.counts + 1, st.pooled_non, p->main));
    if (p->time_fwd[3]) HL_PIPE_TRY(record(p->time_fwd[3], p->main));
    for (auto& t : p->time_fwd) t = nullptr;
    HL_PIPE_TRY(hl_embbag_bwd_apply2(p->ctx, p->cache, st.sorted_slots, st.sorted_bags, st.sorted_n, 1, d_grad_non, lr,
                                     p->main));
    HL_PIPE_TRY(record(e.x, p->main));
    HL_PIPE_TRY(wait(p->wb, e.x));
    HL_PIPE_TRY(hl_scatter_cold_at(p->ctx, p->cache, w0, p->window_rows, st.cold_rows, st.n_cold, p->host_table,
                                   p->wb));
    HL_PIPE_TRY(record(e.scatter, p->wb));
    if (set_index) *set_index = (int32_t)(j % n);
    p->j_done += 1;
    return HL_OK;
}

extern "C" int32_t hl_pipe_time_forward(hl_pipe* p, void* pop_begin, void* pop_end, void* non_begin, void* non_end) {
    if (!p) return HL_EINVAL;
    p->time_fwd[0] = static_cast<cudaEvent_t>(pop_begin);
    p->time_fwd[1] = static_cast<cudaEvent_t>(pop_end);
    p->time_fwd[2] = static_cast<cudaEvent_t>(non_begin);
    p->time_fwd[3] = static_cast<cudaEvent_t>(non_end);
    return HL_OK;
}

extern "C" int32_t hl_pipe_wait_outputs(hl_pipe* p, void* stream) {
    // makes `stream` wait for the last write-back issued (the main stream's own work it sees in order)
    if (!p) return HL_EINVAL;
    if (p->j_done == 0) return HL_OK;
    return wait(static_cast<cudaStream_t>(stream), p->ev[(p->j_done - 1) % p->n_sets].scatter);
}

extern "C" int32_t hl_pipe_wait_counts(hl_pipe* p, void* stream) {
    // perm and counts of the mini-batch last stepped are final once its hl_fragment has run
    if (!p) return HL_EINVAL;
    if (p->j_done == 0) return HL_OK;
    return wait(static_cast<cudaStream_t>(stream), p->ev[(p->j_done - 1) % p->n_sets].frag);
}

extern "C" int32_t hl_pipe_drain(hl_pipe* p) {
    if (!p) return HL_EINVAL;
    cudaStream_t all[6] = {p->main, p->sa, p->sb, p->sc, p->link, p->wb};
    for (auto s : all)
        if (cudaStreamSynchronize(s) != cudaSuccess) return HL_ECUDA;
    return HL_OK;
}
