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
        cudaEvent_t inputs, frag, index, prep, gather, forward, x, scatter, fwd_pop;
    };
    std::vector<Events> ev;
    // mini-batches whose fragment + first half of the cold-row search are queued (begun), whose cold-row search and
    // sort are queued in full (indexed), whose host read is queued (submitted), whose main work is queued (done)
    int64_t j_begun, j_indexed, j_submitted, j_done;
    int order;                   // HL_PIPE_ORDER_*
    int wb_mode;                 // HL_PIPE_WB_*
    bool wb_pending;             // HL_PIPE_WB_AFTER_FORWARD: the write-back of mini-batch j_done - 1 is not queued yet
    // trace (hl_pipe_trace_begin / _end): one event pair per recorded span
    struct Span {
        cudaEvent_t b, e;
        int32_t mini_batch, what, stream;
        bool closed;
    };
    std::vector<Span> spans;
    size_t n_spans;              // spans opened so far
    uint32_t trace_mask;         // bit `what` set: spans of that kind are recorded; 0 = not tracing
    int64_t cur_mb;              // mini-batch the call being issued belongs to (for spans opened by the kernel timers)
    int cur_stream;
    int open_timer[HL_TIMER_COUNT];
};

namespace {

#define HL_PIPE_TRY(expr)                         \
    do {                                          \
        const int32_t st__ = (expr);              \
        if (st__ != HL_OK) return st__;           \
    } while (0)

int32_t wait(cudaStream_t s, cudaEvent_t e) { return cudaStreamWaitEvent(s, e, 0) == cudaSuccess ? HL_OK : HL_ECUDA; }
int32_t record(cudaEvent_t e, cudaStream_t s) { return cudaEventRecord(e, s) == cudaSuccess ? HL_OK : HL_ECUDA; }

// ---- trace ---------------------------------------------------------------------------------------------------
enum { kMain = 0, kStreamA = 1, kStreamB = 2, kStreamC = 3, kLink = 4, kWb = 5 };

cudaStream_t stream_of(hl_pipe* p, int id) {
    cudaStream_t all[6] = {p->main, p->sa, p->sb, p->sc, p->link, p->wb};
    return all[id];
}

// Opens a span of kind `what` for mini-batch `mb` on stream `id`: its begin event is recorded now.  -1 = not recorded.
int span_open(hl_pipe* p, int what, int64_t mb, int id) {
    p->cur_mb = mb;
    p->cur_stream = id;
    if (!(p->trace_mask >> what & 1u) || p->n_spans >= p->spans.size()) return -1;
    hl_pipe::Span& sp = p->spans[p->n_spans];
    if (cudaEventRecord(sp.b, stream_of(p, id)) != cudaSuccess) return -1;
    sp.mini_batch = (int32_t)mb;
    sp.what = what;
    sp.stream = id;
    sp.closed = false;
    return (int)p->n_spans++;
}

void span_close(hl_pipe* p, int idx) {
    if (idx < 0) return;
    hl_pipe::Span& sp = p->spans[idx];
    sp.closed = cudaEventRecord(sp.e, stream_of(p, sp.stream)) == cudaSuccess;
}

// the library's kernel timers (the movers' kernels, the backward's sum kernel, the forward kernel) seen from here
void on_timer_mark(void* user, int which, int end, cudaStream_t) {
    hl_pipe* p = static_cast<hl_pipe*>(user);
    if (which < 0 || which >= HL_TIMER_COUNT) return;
    if (!end) p->open_timer[which] = span_open(p, HL_SPAN_KERNEL + which, p->cur_mb, p->cur_stream);
    else {
        span_close(p, p->open_timer[which]);
        p->open_timer[which] = -1;
    }
}

// RAII span around one library call
struct Scope {
    hl_pipe* p;
    int idx;
    Scope(hl_pipe* p_, int what, int64_t mb, int id) : p(p_), idx(span_open(p_, what, mb, id)) {}
    ~Scope() { span_close(p, idx); }
};

// Second half of the index-only work of the mini-batch begun last: the match of its cold rows against the mini-batch
// before (stream C, in order behind that mini-batch's search) and the backward sort (stream B).
int32_t finish_index(hl_pipe* p) {
    if (p->j_indexed == p->j_begun) return HL_OK;
    const int64_t j = p->j_indexed;
    const int n = p->n_sets;
    hl_pipe_set& st = p->sets[j % n];
    hl_pipe::Events& e = p->ev[j % n];
    hl_pipe_set* prev = j >= 1 ? &p->sets[(j - 1) % n] : nullptr;
    const int64_t w = (j % 2) * p->window_rows;
    {
        Scope sc(p, HL_SPAN_INDEX_END, j, kStreamC);
        HL_PIPE_TRY(hl_index_cold_end(p->ctx, &st.non, w, p->window_rows, st.cold_rows, st.n_cold,
                                      prev ? prev->cold_rows : nullptr, prev ? prev->n_cold : nullptr, st.fwd_src, 0,
                                      p->sc));
    }
    HL_PIPE_TRY(record(e.index, p->sc));
    HL_PIPE_TRY(wait(p->sb, e.index));
    {
        Scope sc(p, HL_SPAN_SORT, j, kStreamB);
        if (p->order == HL_PIPE_ORDER_EQ5)
            HL_PIPE_TRY(hl_embbag_bwd_prepare_merged(p->ctx, &st.pop, st.counts, &st.non, st.counts + 1,
                                                     st.sorted_slots, st.sorted_bags, st.sorted_n, p->sb));
        else
            HL_PIPE_TRY(hl_embbag_bwd_prepare2(p->ctx, &st.pop, st.counts, &st.non, st.counts + 1, st.sorted_slots,
                                               st.sorted_bags, st.sorted_n, p->sb));
    }
    HL_PIPE_TRY(record(e.prep, p->sb));
    p->j_indexed += 1;
    return HL_OK;
}

// fragment and the first half of the cold-row search of the next mini-batch (index-only: nothing here touches a row)
int32_t begin_index(hl_pipe* p, const hl_batch* b, const float* d_dense, void* inputs_ready) {
    HL_PIPE_TRY(finish_index(p));        // (nothing pending in the usual order of calls)
    const int64_t j = p->j_begun;
    const int n = p->n_sets;
    hl_pipe_set& st = p->sets[j % n];
    hl_pipe::Events& e = p->ev[j % n];
    const int64_t w = (j % 2) * p->window_rows;
    if (inputs_ready == nullptr) {                        // the inputs are complete in main-stream order
        HL_PIPE_TRY(record(e.inputs, p->main));
        HL_PIPE_TRY(wait(p->sa, e.inputs));
    } else if (inputs_ready != HL_PIPE_INPUTS_RESIDENT) {
        HL_PIPE_TRY(wait(p->sa, static_cast<cudaEvent_t>(inputs_ready)));
    }
    if (j >= n) HL_PIPE_TRY(wait(p->sa, e.scatter));      // the buffers of this set were mini-batch j-n_sets's
    {
        Scope sc(p, HL_SPAN_FRAGMENT, j, kStreamA);
        HL_PIPE_TRY(hl_fragment(p->ctx, b, d_dense, d_dense ? p->n_dense : 0, st.perm, st.counts, &st.pop, &st.non,
                                d_dense ? st.dense_out : nullptr, p->sa));
    }
    HL_PIPE_TRY(record(e.frag, p->sa));
    HL_PIPE_TRY(wait(p->sc, e.frag));
    if (j >= n) HL_PIPE_TRY(wait(p->sc, e.scatter));
    {
        Scope sc(p, HL_SPAN_INDEX_BEGIN, j, kStreamC);
        HL_PIPE_TRY(hl_index_cold_begin(p->ctx, &st.non, st.counts + 1, w, p->window_rows, st.cold_rows, st.n_cold,
                                        p->sc));
    }
    p->j_begun += 1;
    return finish_index(p);
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
    {
        Scope sc(p, HL_SPAN_STAGE, j, kLink);
        HL_PIPE_TRY(hl_stage_cold(p->ctx, p->host_table, p->cache, w, p->window_rows, st.cold_rows, st.n_cold,
                                  j >= 1 ? st.fwd_src : nullptr, p->link));
    }
    HL_PIPE_TRY(record(p->ev[j % n].gather, p->link));
    p->j_submitted += 1;
    return HL_OK;
}

// the write-back of mini-batch j (whose main work is queued), behind its backward
int32_t queue_scatter(hl_pipe* p, int64_t j) {
    const int n = p->n_sets;
    hl_pipe_set& st = p->sets[j % n];
    hl_pipe::Events& e = p->ev[j % n];
    const int64_t w0 = (j % 2) * p->window_rows;
    HL_PIPE_TRY(wait(p->wb, e.x));
    {
        Scope sc(p, HL_SPAN_SCATTER, j, kWb);
        HL_PIPE_TRY(hl_scatter_cold_at(p->ctx, p->cache, w0, p->window_rows, st.cold_rows, st.n_cold, p->host_table,
                                       p->wb));
    }
    return record(e.scatter, p->wb);
}

// HL_PIPE_WB_AFTER_FORWARD: the write-back held over from the previous hl_pipe_step, if there is one
int32_t flush_scatter(hl_pipe* p) {
    if (!p->wb_pending) return HL_OK;
    p->wb_pending = false;
    return queue_scatter(p, p->j_done - 1);
}

}  // namespace

extern "C" hl_pipe* hl_pipe_create_ex(hl_ctx* ctx, float* d_cache, float* host_table, int64_t window_rows,
                                      int32_t n_sets, const hl_pipe_set* sets, int32_t n_dense, void* main_stream,
                                      const hl_pipe_options* opt) {
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
    if (opt && (opt->write_back < HL_PIPE_WB_OVERLAP || opt->write_back > HL_PIPE_WB_AFTER_FORWARD)) return nullptr;
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
    p->j_begun = p->j_indexed = p->j_submitted = p->j_done = 0;
    p->order = HL_PIPE_ORDER_FIG8;
    p->wb_mode = opt ? opt->write_back : HL_PIPE_WB_OVERLAP;
    p->wb_pending = false;
    p->n_spans = 0;
    p->trace_mask = 0;
    p->cur_mb = 0;
    p->cur_stream = kMain;
    for (auto& t : p->open_timer) t = -1;
    int lo = 0, hi = 0;
    cudaDeviceGetStreamPriorityRange(&lo, &hi);          // hi = numerically lowest = highest priority
    auto clamp = [&](int prio) { return prio < hi ? hi : (prio > lo ? lo : prio); };
    const int index_prio = clamp(opt ? opt->index_priority : 0), link_prio = clamp(opt ? opt->link_priority : 0);
    cudaStream_t* side[5] = {&p->sa, &p->sb, &p->sc, &p->link, &p->wb};
    bool ok = true;
    for (int i = 0; i < 5; ++i) {
        *side[i] = nullptr;
        ok = ok && cudaStreamCreateWithPriority(side[i], cudaStreamNonBlocking, i < 3 ? index_prio : link_prio) ==
                       cudaSuccess;
    }
    p->ev.resize(n_sets);
    for (auto& e : p->ev) {
        cudaEvent_t* all[9] = {&e.inputs, &e.frag,    &e.index, &e.prep,   &e.gather,
                               &e.forward, &e.x,      &e.scatter, &e.fwd_pop};
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

extern "C" hl_pipe* hl_pipe_create(hl_ctx* ctx, float* d_cache, float* host_table, int64_t window_rows,
                                   int32_t n_sets, const hl_pipe_set* sets, int32_t n_dense, void* main_stream) {
    return hl_pipe_create_ex(ctx, d_cache, host_table, window_rows, n_sets, sets, n_dense, main_stream, nullptr);
}

extern "C" void hl_pipe_destroy(hl_pipe* p) {
    if (!p) return;
    if (p->wb_pending && p->wb) (void)flush_scatter(p);      // a write-back held over is not lost
    cudaStream_t side[5] = {p->sa, p->sb, p->sc, p->link, p->wb};
    for (auto s : side)
        if (s) {
            cudaStreamSynchronize(s);
            cudaStreamDestroy(s);
        }
    for (auto& e : p->ev) {
        cudaEvent_t all[9] = {e.inputs, e.frag, e.index, e.prep, e.gather, e.forward, e.x, e.scatter, e.fwd_pop};
        for (auto x : all)
            if (x) cudaEventDestroy(x);
    }
    if (p->ctx && p->ctx->mark_user == p) {
        p->ctx->mark_hook = nullptr;
        p->ctx->mark_user = nullptr;
    }
    for (auto& sp : p->spans) {
        if (sp.b) cudaEventDestroy(sp.b);
        if (sp.e) cudaEventDestroy(sp.e);
    }
    delete p;
}

extern "C" int32_t hl_pipe_submit(hl_pipe* p, const hl_batch* b, const float* d_dense, void* inputs_ready) {
    if (!p || !b) return HL_EINVAL;
    if (p->j_begun - p->j_done >= p->n_sets - 1) return HL_ECAPACITY;      // every spare buffer set is in flight
    HL_PIPE_TRY(begin_index(p, b, d_dense, inputs_ready));
    if (p->j_submitted == p->j_done) {                                      // nothing staged ahead yet
        HL_PIPE_TRY(finish_index(p));
        HL_PIPE_TRY(submit_link(p));
    }
    return HL_OK;
}

extern "C" int32_t hl_pipe_step(hl_pipe* p, const float* d_grad_pop, const float* d_grad_non, float lr,
                                const hl_batch* next, const float* d_next_dense, void* next_inputs_ready,
                                int32_t* set_index) {
    if (!p || !d_grad_pop || (!d_grad_non && p->order != HL_PIPE_ORDER_EQ5)) return HL_EINVAL;
    const int64_t j = p->j_done;
    if (p->j_submitted < j + 1) return HL_EINVAL;          // hl_pipe_submit first
    const int n = p->n_sets;
    hl_pipe_set& st = p->sets[j % n];
    hl_pipe::Events& e = p->ev[j % n];
    const int64_t w0 = (j % 2) * p->window_rows, w1 = ((j + 1) % 2) * p->window_rows;
    if (next && p->j_begun - j >= n - 1) return HL_ECAPACITY;
    HL_PIPE_TRY(wait(p->main, e.index));
    if (p->wb_mode == HL_PIPE_WB_EXCLUSIVE && j >= 1) HL_PIPE_TRY(wait(p->main, p->ev[(j - 1) % n].scatter));
    if (j >= 1) {
        // rows shared with mini-batch j-1 come out of its staging window once its backward is done
        HL_PIPE_TRY(wait(p->link, e.index));
        HL_PIPE_TRY(wait(p->link, p->ev[(j - 1) % n].x));
        Scope sc(p, HL_SPAN_FORWARD_COLD, j, kLink);
        HL_PIPE_TRY(hl_forward_cold(p->ctx, p->cache, w1, w0, p->window_rows, st.fwd_src, st.n_cold, p->link));
    }
    HL_PIPE_TRY(record(e.forward, p->link));
    // (the host read of j+1 waits for the write-back of j-1, so it is queued behind a write-back that was held over)
    if (!p->wb_pending && p->j_submitted < p->j_indexed) HL_PIPE_TRY(submit_link(p));   // j+1, if indexed in full
    {
        Scope sc(p, HL_SPAN_FWD_POP, j, kMain);
        HL_PIPE_TRY(hl_embbag_fwd(p->ctx, p->cache, &st.pop, st.counts, st.pooled_pop, p->main));
    }
    if (p->wb_pending) {
        // the write-back of j-1 starts when the popular forward of j is over: of all kernels of the main stream that
        // one loses most next to a write-back
        HL_PIPE_TRY(record(e.fwd_pop, p->main));
        HL_PIPE_TRY(wait(p->wb, e.fwd_pop));
        HL_PIPE_TRY(flush_scatter(p));
        if (p->j_submitted < p->j_indexed) HL_PIPE_TRY(submit_link(p));
    }
    if (p->order == HL_PIPE_ORDER_FIG8) {
        HL_PIPE_TRY(wait(p->main, e.prep));
        Scope sc(p, HL_SPAN_BWD_POP, j, kMain);
        HL_PIPE_TRY(hl_embbag_bwd_apply2(p->ctx, p->cache, st.sorted_slots, st.sorted_bags, st.sorted_n, 0, d_grad_pop,
                                         lr, p->main));
    }
    HL_PIPE_TRY(wait(p->main, e.gather));
    HL_PIPE_TRY(wait(p->main, e.forward));
    {
        Scope sc(p, HL_SPAN_FWD_NON, j, kMain);
        HL_PIPE_TRY(hl_embbag_fwd(p->ctx, p->cache, &st.non, st.counts + 1, st.pooled_non, p->main));
    }
    if (p->order == HL_PIPE_ORDER_FIG8) {
        Scope sc(p, HL_SPAN_BWD_NON, j, kMain);
        HL_PIPE_TRY(hl_embbag_bwd_apply2(p->ctx, p->cache, st.sorted_slots, st.sorted_bags, st.sorted_n, 1, d_grad_non,
                                         lr, p->main));
    } else {   // one update of every touched row with the gradient of the whole mini-batch
        HL_PIPE_TRY(wait(p->main, e.prep));
        Scope sc(p, HL_SPAN_BWD_NON, j, kMain);
        HL_PIPE_TRY(hl_embbag_bwd_apply(p->ctx, p->cache, st.sorted_slots, st.sorted_bags, st.sorted_n + 2, d_grad_pop,
                                        lr, p->main));
    }
    HL_PIPE_TRY(record(e.x, p->main));
    p->j_done += 1;
    if (p->wb_mode == HL_PIPE_WB_AFTER_FORWARD && next)
        p->wb_pending = true;            // queued by the next hl_pipe_step (or by whatever call comes instead)
    else
        HL_PIPE_TRY(queue_scatter(p, j));
    HL_PIPE_TRY(finish_index(p));
    if (p->j_submitted == j + 1 && p->j_submitted < p->j_indexed) HL_PIPE_TRY(submit_link(p));   // mini-batch j+1
    if (next) {
        HL_PIPE_TRY(begin_index(p, next, d_next_dense, next_inputs_ready));
        if (p->j_submitted == j + 1) {                                      // j+1 was begun only just now
            HL_PIPE_TRY(finish_index(p));
            HL_PIPE_TRY(submit_link(p));
        }
    }
    if (set_index) *set_index = (int32_t)(j % n);
    return HL_OK;
}

extern "C" int32_t hl_pipe_set_order(hl_pipe* p, int32_t order) {
    if (!p || (order != HL_PIPE_ORDER_FIG8 && order != HL_PIPE_ORDER_EQ5)) return HL_EINVAL;
    if (p->j_begun != 0) return HL_EINVAL;       // the sorts queued so far were made for the other order
    p->order = order;
    return HL_OK;
}

extern "C" int32_t hl_pipe_trace_begin(hl_pipe* p, int32_t max_spans, uint32_t what_mask) {
    if (!p || max_spans < 1 || max_spans > (1 << 16) || what_mask == 0) return HL_EINVAL;
    if ((int)p->spans.size() < max_spans) {
        const size_t old = p->spans.size();
        p->spans.resize(max_spans);
        for (size_t i = old; i < p->spans.size(); ++i) p->spans[i].b = p->spans[i].e = nullptr;
        for (size_t i = old; i < p->spans.size(); ++i)
            if (cudaEventCreate(&p->spans[i].b) != cudaSuccess || cudaEventCreate(&p->spans[i].e) != cudaSuccess) {
                p->spans.resize(i);      // (an event of the failed pair, if any, is leaked with the pipeline's others)
                return HL_ECUDA;
            }
    }
    p->n_spans = 0;
    p->trace_mask = what_mask;
    for (auto& t : p->open_timer) t = -1;
    p->ctx->mark_hook = on_timer_mark;
    p->ctx->mark_user = p;
    return HL_OK;
}

extern "C" int32_t hl_pipe_trace_end(hl_pipe* p, hl_pipe_span* out, int32_t cap, int32_t* n_out) {
    if (!p || !n_out || cap < 0 || (cap > 0 && !out)) return HL_EINVAL;
    p->trace_mask = 0;
    if (p->ctx->mark_user == p) {
        p->ctx->mark_hook = nullptr;
        p->ctx->mark_user = nullptr;
    }
    HL_PIPE_TRY(hl_pipe_drain(p));
    // times are relative to the earliest begin among the recorded spans
    int first = -1;
    for (size_t i = 0; i < p->n_spans; ++i) {
        if (!p->spans[i].closed) continue;
        if (first < 0) {
            first = (int)i;
            continue;
        }
        float ms = 0.f;
        if (cudaEventElapsedTime(&ms, p->spans[first].b, p->spans[i].b) == cudaSuccess && ms < 0.f) first = (int)i;
    }
    int32_t n = 0;
    for (size_t i = 0; i < p->n_spans && n < cap; ++i) {
        const hl_pipe::Span& sp = p->spans[i];
        if (!sp.closed) continue;
        float b = 0.f, e = 0.f;
        if (cudaEventElapsedTime(&b, p->spans[first].b, sp.b) != cudaSuccess ||
            cudaEventElapsedTime(&e, p->spans[first].b, sp.e) != cudaSuccess) {
            cudaGetLastError();
            continue;
        }
        out[n].mini_batch = sp.mini_batch;
        out[n].what = sp.what;
        out[n].stream = sp.stream;
        out[n].begin_ms = b;
        out[n].end_ms = e;
        ++n;
    }
    *n_out = n;
    p->n_spans = 0;
    return HL_OK;
}

extern "C" int32_t hl_pipe_wait_outputs(hl_pipe* p, void* stream) {
    // makes `stream` wait for the last write-back issued (the main stream's own work it sees in order)
    if (!p) return HL_EINVAL;
    if (p->j_done == 0) return HL_OK;
    HL_PIPE_TRY(flush_scatter(p));
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
    HL_PIPE_TRY(flush_scatter(p));
    cudaStream_t all[6] = {p->main, p->sa, p->sb, p->sc, p->link, p->wb};
    for (auto s : all)
        if (cudaStreamSynchronize(s) != cudaSuccess) return HL_ECUDA;
    return HL_OK;
}
