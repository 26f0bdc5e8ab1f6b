/*
 * hotline.h -- C boundary of the B200 (sm_100a) library for the data-parallel hot path of the Hotline
 * heterogeneous embedding pipeline (arXiv 2204.05436).
 *
 * The path, per mini-batch (paper Section IV "Acceleration Phase", Fig. 8):
 *   hl_fragment        split mini-batch M into the popular micro-batch O (every lookup hits a popular row)
 *                      and the non-popular micro-batch X                              (Sections I, V-A, V-C; Eq. 3)
 *   hl_gather_cold     stage X's non-popular working rows from the host-DRAM table behind the hot cache,
 *                      on a side stream, while O executes                              (Sections IV, V-A)
 *   hl_embbag_fwd      sum-pool the rows of every bag                                 (the Reducer, Section V-D)
 *   hl_embbag_bwd_sgd  scatter-add the pooled gradients per distinct row, one SGD update per row (Section IV)
 *   hl_scatter_cold    write X's updated cold rows back to the host table              (Section IV, dma_wr)
 * and, once per learning phase (Section IV "Learning Phase", Section V-B):
 *   hl_profile_hot     count row accesses over sampled mini-batches and select the popular rows
 *   hl_build_remap     build the popular-row lookup structure and load the popular rows into HBM.
 *
 * Conventions
 *   - Pointers named d_* are DEVICE pointers (16-byte aligned); h_* are HOST pointers; `host_table` must be
 *     readable/writable from the device (pinned, mapped host memory; device memory also works).
 *   - The caller owns every buffer.  The library allocates nothing on the device: its scratch lives in the
 *     caller-provided workspace given to hl_create (size from hl_workspace_bytes).
 *   - Every call returns an int32 status (HL_OK = 0, negative = error) for what the host can check.  Calls are
 *     asynchronous on `stream` (a cudaStream_t passed as void*); errors found on the device (an index outside
 *     its table, a capacity overflow) never trap: the offending item is skipped, a status word is set, and
 *     hl_status() returns it.
 *   - No call synchronises the host, so sizes that depend on the data (number of popular inputs, number of
 *     cold rows, lookups per micro-batch) stay in device memory and are passed between calls as pointers.
 *   - Mini-batch layout: table-major CSR.  Bag beta(t, b, s) = (t*B + b)*S + s for table t, input b, step s
 *     holds indices[offsets[beta] .. offsets[beta+1]), table-local int32 row ids.  Global row id
 *     g = base_t + index, base_t = rows of all earlier tables.  N = total rows < 2^31.
 *   - fp32 values; dim % 4 == 0.
 *   - Calls that share a context may overlap on different streams only as stated per call (each call names
 *     the scratch region it uses).
 */
#ifndef HOTLINE_H_
#define HOTLINE_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#if defined(__GNUC__)
#define HL_API __attribute__((visibility("default")))
#else
#define HL_API
#endif

#define HL_OK          0
#define HL_EINVAL    (-1)   /* bad argument, shape or alignment (host check), or malformed device data          */
#define HL_EBOUNDS   (-2)   /* an index outside its table / a slot outside the cache (device; item skipped)      */
#define HL_ECAPACITY (-3)   /* an output buffer, the hot cache or the staging area is too small (device; clamped)*/
#define HL_ECUDA     (-4)   /* a CUDA runtime call failed                                                        */
#define HL_ETIMEOUT  (-5)   /* a bounded device-side wait (tile chaining of a scan or sort, a bulk copy) gave up  */

typedef struct hl_ctx hl_ctx;

/* Model geometry.  table_rows is a HOST array of num_tables row counts. */
typedef struct {
    int32_t        num_tables;       /* T                                                         */
    int32_t        dim;              /* D, fp32 columns per row, multiple of 4                    */
    int32_t        bags_per_sample;  /* S: bags per input and table (21 time steps, else 1)       */
    const int64_t* table_rows;       /* host, [T]                                                 */
} hl_geometry;

/* One mini-batch in device memory (table-major CSR, see above). */
typedef struct {
    const int32_t* indices;          /* device, [nnz]                                             */
    const int32_t* offsets;          /* device, [T*batch*S + 1], offsets[0] = 0                   */
    int32_t        batch;            /* B inputs                                                  */
    int64_t        nnz;              /* total lookups L = offsets[T*batch*S]                      */
} hl_batch;

/* One micro-batch in device memory, caller-sized for the worst case (all inputs land in it). */
typedef struct {
    int32_t* offsets;                /* device, [T*max_batch*S + 1]                               */
    int32_t* ids;                    /* device, [cap_ids]: cache slots, or global rows (X before hl_gather_cold) */
    int64_t  cap_ids;
} hl_ubatch;

/* How hl_profile_hot turns counts into a popular set.  All policies rank rows seen at least once by
 * (count descending, global id ascending), one ranking across all tables, and clip to the hot capacity. */
enum {
    HL_HOT_TOPK_ROWS     = 0,        /* keep p_num rows                                           */
    HL_HOT_BUDGET_BYTES  = 1,        /* keep floor(p_num / (4*D)) rows (row payload only)         */
    HL_HOT_FRACTION_ROWS = 2,        /* keep floor(N * p_num / p_den) rows                        */
    HL_HOT_MIN_SHARE     = 3         /* keep rows with count/total >= p_num/p_den (the paper's
                                        1-in-100,000 criterion, Fig. 4), exact integer test       */
};

/* ---------------------------------------------------------------------------------------------------------
 * Support calls (no counterpart in the paper; they carry the address registers of the Data Dispatcher,
 * Section V-A: one base per table).
 * ------------------------------------------------------------------------------------------------------- */

/* Bytes of device workspace a context needs for mini-batches of at most max_batch inputs and max_nnz
 * lookups, hot_cap_rows cache slots and staging_cap_rows staging slots.  0 on invalid arguments. */
HL_API size_t hl_workspace_bytes(const hl_geometry* geom, int32_t max_batch, int64_t max_nnz,
                          int64_t hot_cap_rows, int64_t staging_cap_rows);

/* Creates a context on the current device.  d_workspace (device, 256-byte aligned, ws_bytes long) stays
 * owned by the caller and must outlive the context.  Synchronous (initialises the workspace).
 * The cache the other calls take is fp32 [(hot_cap_rows + staging_cap_rows), D]: slots [0, hot_cap_rows) hold
 * popular rows, slot hot_cap_rows + i holds the i-th staged cold row. */
HL_API int32_t hl_create(hl_ctx** out, const hl_geometry* geom, int32_t max_batch, int64_t max_nnz,
                  int64_t hot_cap_rows, int64_t staging_cap_rows, void* d_workspace, size_t ws_bytes);
HL_API int32_t hl_destroy(hl_ctx* ctx);

/* Synchronises the device, returns the first device-side error recorded since the last call (HL_OK if
 * none) and clears it. */
HL_API int32_t hl_status(hl_ctx* ctx);

HL_API const char* hl_strerror(int32_t status);

/* Optional kernel timers, off by default.  When enabled, the library records a CUDA event pair on the call's
 * stream around: the row-move kernel of hl_gather_cold (HL_TIMER_GATHER_MOVE) and of hl_scatter_cold
 * (HL_TIMER_SCATTER_MOVE), the segment-reduce + update kernel of hl_embbag_bwd_sgd (HL_TIMER_BWD_REDUCE), the
 * kernel of hl_embbag_fwd (HL_TIMER_FWD).  hl_timing_read gives the milliseconds of the LAST recorded pair; the
 * caller synchronises first (HL_EINVAL if the pair was never recorded or has not finished). */
#define HL_TIMER_GATHER_MOVE  0
#define HL_TIMER_SCATTER_MOVE 1
#define HL_TIMER_BWD_REDUCE   2
#define HL_TIMER_FWD          3
#define HL_TIMER_COUNT        4
HL_API int32_t hl_timing_enable(hl_ctx* ctx, int32_t on);
HL_API int32_t hl_timing_read(hl_ctx* ctx, int32_t which, float* ms);

/* Host-resident, device-mapped memory for the host-DRAM table (exactly `bytes`): the current device reads and
 * writes it in place over the host link, at the same address the CPU uses; the pages stay in host DRAM.  (Unified
 * memory with the CPU as preferred location and the device advised to map it, which the device maps in large pages;
 * memory from cudaHostAlloc also works as a table but is mapped in 4 KB pages, and random rows of a table of tens of
 * GB then pay an address-translation miss each.  If unified memory refuses the size -- on the bench platform a single
 * allocation stops between 66 and 70 GB -- the call falls back to such memory; a larger table is better held as one
 * allocation per table, see hl_set_host_tables.)  The caller owns it and frees it with hl_host_free.  Returns NULL on
 * failure. */
HL_API void* hl_host_alloc(size_t bytes);
HL_API int32_t hl_host_free(void* p);

/* Section V-A (the Data Dispatcher keeps one base address per table).  Installs one host-memory allocation per
 * table instead of a single allocation that holds all tables back to back: h_table_bases is a HOST array of
 * num_tables pointers, each to fp32 [table_rows[t], D] that the device can read and write (16-byte aligned).  From
 * then on global row g of table t is at h_table_bases[t] + (g - base_t) * D, and the `host_table` argument of every
 * other call only says whether the host table takes part (non-NULL) -- its value is not used.  NULL returns to the
 * single-allocation form.  Synchronises the device.  (A table too large for one allocation of hl_host_alloc's
 * large-page memory -- 8 x 9.5 GiB of the multi-hot configuration, say -- is held this way.) */
HL_API int32_t hl_set_host_tables(hl_ctx* ctx, float* const* h_table_bases);

/* Width of the host-link movers inside a schedule: how many CTAs of hl_gather_cold / hl_stage_cold (read_ctas) and of
 * hl_scatter_cold (write_ctas) work when a mini-batch moves a DLRM-sized number of rows (the kernels decide on the
 * device, from the number of rows, whether more join in).  0 = the default (24 for reads, 16 for write-backs); at
 * most two per multiprocessor.  Wider movers finish sooner and slow the kernels that run beside them more.  Takes
 * effect with the next call. */
HL_API int32_t hl_set_mover_ctas(hl_ctx* ctx, int32_t read_ctas, int32_t write_ctas);

/* Grid size of the two bandwidth-bound kernels, in CTAs per multiprocessor: the forward kernel (hl_embbag_fwd) and
 * the backward's sum kernel (hl_embbag_bwd_*).  Both deal their work out evenly over a fixed grid; fewer CTAs per
 * multiprocessor leave registers and shared memory for the kernels of other streams (index work, movers) to run
 * beside them, more give the kernel itself more loads in flight.  0 = the default (4 for the forward, 3 for rows wider
 * than 128 fp32; 6 for the sum kernel). */
HL_API int32_t hl_set_kernel_width(hl_ctx* ctx, int32_t fwd_ctas_per_sm, int32_t bwd_ctas_per_sm);

/* Test aid for the bounded device-side waits (the tile chaining of the scan inside hl_fragment and of the sorts
 * inside hl_embbag_bwd_* / hl_gather_cold, the wait of a row mover for a stage of bulk copies).  In production these
 * waits poll for about a second before they give up, which never happens.  poll_limit > 0 makes them give up after
 * that many polls, and makes ONE participant withhold what the others wait for: tile `stall_tile` of every chained scan
 * and sort pass publishes nothing, and (stall_tile >= 0) the first stage of the movers' first CTA issues no copies.
 * The waits behind it then run out: the kernels return, the status word reads HL_ETIMEOUT, every position computed
 * from the incomplete data is range-checked before use, and the results of those calls are unspecified.
 * poll_limit = 0 restores production behaviour.  Nothing here can hang or fault the device. */
HL_API int32_t hl_test_bounded_waits(hl_ctx* ctx, int32_t poll_limit, int64_t stall_tile);

/* Number of kernels this library has launched from the host in this process so far (all contexts; the general cold-row
 * search that a kernel launches from the device is not counted). */
HL_API uint64_t hl_launch_count(void);

/* ---------------------------------------------------------------------------------------------------------
 * Learning phase
 * ------------------------------------------------------------------------------------------------------- */

/* Section IV "Learning Phase" / Section V-B (the exact counter the paper calls the Oracle LFU logger).
 * If reset != 0 the per-row access counters are cleared first.  If b != NULL every lookup of the mini-batch
 * adds one to its row's counter (repeats inside a bag count again).  If finalize != 0 the popular rows are
 * selected by `policy` (see the enum) and written in ASCENDING global id to d_hot_rows [hot_cap_rows], their
 * number to *d_n_hot.  Scratch: the profile region.  Must not overlap with other calls on this context. */
HL_API int32_t hl_profile_hot(hl_ctx* ctx, const hl_batch* b, int32_t reset, int32_t finalize,
                       int32_t policy, int64_t p_num, int64_t p_den,
                       int32_t* d_hot_rows, int64_t* d_n_hot, void* stream);

/* Section V-B "Efficient Embedding Tracking" (the access logger as the paper builds it) with the randomizer of
 * Section V-C: a set-associative table of n_sets x ways blocks, each a row tag (global row id, -1 = empty) and a
 * 2-bit re-reference prediction value (RRPV), replaced by SRRIP: a hit sets the block's RRPV to 0; a miss takes the
 * first way, from way 0, whose RRPV is 3 (empty ways hold 3), incrementing every RRPV of the set until there is one,
 * and inserts the row with RRPV 2.  A row's set is randomizer(row) mod n_sets, the randomizer a 4-round Feistel
 * network on the 16-bit halves of the row id with round function F_r(x) = upper 16 bits of
 * (x * 0x9E3779B1 + K_r) mod 2^32, K = {0x85EBCA6B, 0xC2B2AE35, 0x27D4EB2F, 0x165667B1}.  (The paper fixes the
 * policy, the counter width and the insertion value; associativity, victim order and the rounds are this library's.)
 * The state lives in caller-owned device arrays d_tags [n_sets*ways] int32 and d_rrpv [n_sets*ways] uint8
 * (1 <= ways <= 32); d_hits (may be NULL) accumulates the number of hits.
 *
 * hl_tracker_reset   empties the logger (and clears *d_hits).
 * hl_tracker_update  presents every lookup of the mini-batch to the logger; the result is that of serving them one
 *                    after the other in the order of the layout (position 0 .. nnz-1 of `indices`).  Lookups outside
 *                    their table are skipped (HL_EBOUNDS).  Scratch: the backward region.
 * hl_tracker_export  writes what the logger holds into the context's access counters -- counter = 4 - RRPV for a
 *                    tracked row, 0 for every other row -- after which hl_profile_hot(b = NULL, reset = 0,
 *                    finalize = 1, ...) selects the popular rows among the tracked ones by its usual rules (all of
 *                    them if the capacity allows, the most recently re-referenced first otherwise).
 * None of the three may overlap with other calls on this context. */
HL_API int32_t hl_tracker_reset(hl_ctx* ctx, int32_t* d_tags, uint8_t* d_rrpv, int64_t n_sets, int32_t ways,
                                unsigned long long* d_hits, void* stream);
HL_API int32_t hl_tracker_update(hl_ctx* ctx, const hl_batch* b, int32_t* d_tags, uint8_t* d_rrpv, int64_t n_sets,
                                 int32_t ways, unsigned long long* d_hits, void* stream);
HL_API int32_t hl_tracker_export(hl_ctx* ctx, const int32_t* d_tags, const uint8_t* d_rrpv, int64_t n_sets,
                                 int32_t ways, void* stream);

/* Section IV: popular rows are replicated in GPU memory, the classifier keeps only their indices.
 * Builds the lookup structure for the popular set d_hot_rows[0 .. *d_n_hot) (strictly ascending global ids;
 * any such set is allowed, misclassification never affects fidelity): the cache slot of a popular row is its
 * rank in that list.  If host_table != NULL also loads cache[i, :] = host_table[hot_rows[i], :] (bit copy).
 * If d_remap_out != NULL writes the dense map remap[g] = slot or -1, int32 [N].
 * Must not overlap with other calls on this context. */
HL_API int32_t hl_build_remap(hl_ctx* ctx, const int32_t* d_hot_rows, const int64_t* d_n_hot,
                       const float* host_table, float* d_cache, int32_t* d_remap_out, void* stream);

/* Section V-B (the logger periodically returns to its learning phase to follow changes in popularity) and
 * Section IV (popular rows live in GPU memory only): before a new popular set replaces the current one, the
 * current values of the popular rows go back to the host table:
 * host_table[d_hot_rows[i], :] = cache[i, :] for i < *d_n_hot.  Afterwards the host table holds every row's
 * current value (a consistent snapshot), and hl_profile_hot / hl_build_remap may install another set. */
HL_API int32_t hl_flush_hot(hl_ctx* ctx, const float* d_cache, const int32_t* d_hot_rows, const int64_t* d_n_hot,
                            float* host_table, void* stream);

/* ---------------------------------------------------------------------------------------------------------
 * Acceleration phase
 * ------------------------------------------------------------------------------------------------------- */

/* Sections I, V-A (Input Classifier), V-C (Lookup Engine), Eq. 3.
 * An input is popular iff every lookup of it, over all tables and steps, addresses a popular row (an input
 * without lookups is popular).  Outputs:
 *   d_perm   [B]   inputs of O in ascending order, then inputs of X in ascending order
 *   d_counts [4]   { n_pop, n_non, lookups in O, lookups in X }
 *   pop            O as table-major CSR over its n_pop inputs; ids = cache slots
 *   non            X as table-major CSR over its n_non inputs; ids = GLOBAL row ids (-1 for an index that was
 *                  outside its table: such a lookup counts as a miss and is ignored downstream)
 *   d_dense_out    optional [B, n_dense]: d_dense rows in d_perm order (values untouched)
 * Scratch: the fragment region (may overlap with embbag/cold calls of an earlier mini-batch). */
HL_API int32_t hl_fragment(hl_ctx* ctx, const hl_batch* b, const float* d_dense, int32_t n_dense,
                    int32_t* d_perm, int32_t* d_counts, hl_ubatch* pop, hl_ubatch* non,
                    float* d_dense_out, void* stream);

/* Section V-D (Reducer: sparse-length element-wise sum).
 * out[beta, :] = sum over the bag's lookups of cache[ids[j], :], for the T * (*d_n_samples) * S bags of the
 * micro-batch; an empty bag gives zeros; negative ids are skipped.  d_out is [T*max_batch*S, D].
 * Uses no scratch: may overlap with anything that does not write the rows it reads. */
HL_API int32_t hl_embbag_fwd(hl_ctx* ctx, const float* d_cache, const hl_ubatch* ub, const int32_t* d_n_samples,
                      float* d_out, void* stream);

/* Section IV (popular rows are updated in GPU memory; plain SGD as the optimizer).
 * For every distinct id u of the micro-batch: G_u = sum over lookups j with ids[j] == u of
 * d_grad_out[bag(j), :], then cache[u, :] -= lr * G_u, exactly one read-modify-write per row and call: the lookups
 * are sorted by id, every run of equal ids is summed in a fixed order, and -(lr * G_u) is added to the row by one
 * reduction (red.global.add.f32) per element.  With a single addition per element and call the result does not depend
 * on the order in which rows are served, so the call is deterministic.  Rows not referenced keep their bits.
 * Scratch: the backward region (may overlap with hl_gather_cold / hl_fragment, not with itself). */
HL_API int32_t hl_embbag_bwd_sgd(hl_ctx* ctx, float* d_cache, const hl_ubatch* ub, const int32_t* d_n_samples,
                          const float* d_grad_out, float lr, void* stream);

/* The two halves of hl_embbag_bwd_sgd as separate calls.  hl_embbag_bwd_prepare does the part that depends only on
 * the micro-batch's ids: the (slot, bag) pair of every lookup, stably sorted by slot, into d_sorted_slots /
 * d_sorted_bags [cap_ids each], their number into *d_n_lookups.  It can therefore run ahead, on another stream, as
 * soon as the ids are final (for X: after hl_gather_cold / hl_index_cold), which takes the sort off the path between
 * a forward and its backward.  hl_embbag_bwd_apply then sums the gradient rows per run of equal slots and applies the
 * one SGD update per row.  Scratch: prepare uses the sort buffers of the backward region (as hl_embbag_bwd_sgd does:
 * do not overlap two of them), apply the partial-sum buffer of the backward region (do not overlap two applies). */
HL_API int32_t hl_embbag_bwd_prepare(hl_ctx* ctx, const hl_ubatch* ub, const int32_t* d_n_samples,
                                     int32_t* d_sorted_slots, int32_t* d_sorted_bags, int32_t* d_n_lookups,
                                     void* stream);
HL_API int32_t hl_embbag_bwd_apply(hl_ctx* ctx, float* d_cache, const int32_t* d_sorted_slots,
                                   const int32_t* d_sorted_bags, const int32_t* d_n_lookups, const float* d_grad_out,
                                   float lr, void* stream);

/* One sort for both micro-batches of a mini-batch: hl_embbag_bwd_prepare2 sorts the (slot, bag) pairs of O and X
 * together (X's keys offset by the number of cache slots + 1, so that O's pairs come first, a skipped lookup of O,
 * negative id, last among them), which costs one three-pass sort instead of two; d_n_lookups[0..2] = lookups of O,
 * lookups of X, their sum.
 * hl_embbag_bwd_apply2(which = 0 for O, 1 for X) is hl_embbag_bwd_apply on that micro-batch's part of the arrays.
 * d_sorted_slots / d_sorted_bags hold cap_ids(pop) + cap_ids(non) <= max_nnz entries.  Scratch as for prepare / apply. */
HL_API int32_t hl_embbag_bwd_prepare2(hl_ctx* ctx, const hl_ubatch* pop, const int32_t* d_n_pop, const hl_ubatch* non,
                                      const int32_t* d_n_non, int32_t* d_sorted_slots, int32_t* d_sorted_bags,
                                      int32_t* d_n_lookups, void* stream);
HL_API int32_t hl_embbag_bwd_apply2(hl_ctx* ctx, float* d_cache, const int32_t* d_sorted_slots,
                                    const int32_t* d_sorted_bags, const int32_t* d_n_lookups, int32_t which,
                                    const float* d_grad_out, float lr, void* stream);

/* Section IV-A, Eq. 5 (the two micro-batches together give the mini-batch's gradient): hl_embbag_bwd_prepare_merged
 * sorts the pairs of O and X in ONE key space, X's bags numbered behind O's, so that all lookups of a row, from either
 * micro-batch, form one run.  hl_embbag_bwd_apply(ctx, cache, slots, bags, d_n_lookups + 2, d_grad_all, lr, stream) on
 * the result, with d_grad_all = [gradients of O's bags; gradients of X's bags] (X's block starts at row
 * T * (*d_n_pop) * S), then updates every row once with the whole mini-batch's gradient -- the result of the
 * unfragmented step when both forwards ran before it.  Same arguments and scratch as hl_embbag_bwd_prepare2. */
HL_API int32_t hl_embbag_bwd_prepare_merged(hl_ctx* ctx, const hl_ubatch* pop, const int32_t* d_n_pop,
                                            const hl_ubatch* non, const int32_t* d_n_non, int32_t* d_sorted_slots,
                                            int32_t* d_sorted_bags, int32_t* d_n_lookups, void* stream);

/* Sections IV and V-A (dma_rd of non-popular rows; popular rows of X are read from GPU memory).
 * In:  non->ids = global rows of X (from hl_fragment), *d_n_non = inputs in X.
 * Out: d_cold_rows[0 .. *d_n_cold) = the distinct non-popular rows referenced by X, ascending (each staged
 *      once); non->ids rewritten to unified cache slots (hot slot, or hot_cap_rows + rank in d_cold_rows);
 *      cache[hot_cap_rows + i, :] = host_table[d_cold_rows[i], :].
 * Touches only the staging part of the cache: may run on a side stream while O's forward/backward run.
 * Scratch: the cold region. */
HL_API int32_t hl_gather_cold(hl_ctx* ctx, hl_ubatch* non, const int32_t* d_n_non, const float* host_table,
                       float* d_cache, int32_t* d_cold_rows, int64_t* d_n_cold, void* stream);

/* Section IV (non-popular rows are updated in CPU memory by DMA write).
 * host_table[d_cold_rows[i], :] = cache[hot_cap_rows + i, :] for i < *d_n_cold.  No scratch. */
HL_API int32_t hl_scatter_cold(hl_ctx* ctx, const float* d_cache, const int32_t* d_cold_rows,
                        const int64_t* d_n_cold, float* host_table, void* stream);

/* ---------------------------------------------------------------------------------------------------------
 * Software pipelining across mini-batches (Section IV: the gathering of the working parameters is pipelined with
 * the execution on the GPU so that the GPU never stalls).  While mini-batch j-1 is still executing, mini-batch j
 * can already be fragmented and its cold rows staged, provided that a cold row which j shares with j-1 is NOT
 * read from the host (its update by j-1 has not been written back yet) but copied from j-1's staging area once
 * j-1's backward has run.  The staging part of the cache is used as several windows (stage_row0, stage_rows):
 * a row of rank r is staged at cache slot hot_cap_rows + stage_row0 + r.
 * ------------------------------------------------------------------------------------------------------- */

/* hl_gather_cold into the window [stage_row0, stage_row0 + stage_rows) of the staging area, with exclusion:
 * d_prev_cold_rows[0 .. *d_n_prev) (ascending; may be NULL) is the cold set of the mini-batch still in flight.
 * d_fwd_src[i] (out, [stage_rows]) = position of d_cold_rows[i] in that set, or -1; rows with d_fwd_src[i] >= 0
 * are not read from the host (hl_forward_cold fills them in later).
 * Optional CUDA events (cudaEvent_t as void*, may be NULL): record_after_index is recorded on the stream once
 * d_cold_rows, *d_n_cold, d_fwd_src and the unified slots in non->ids are final; the stream waits for
 * wait_before_move_a / _b right before the host rows are read (e.g. the write-back of an earlier mini-batch). */
HL_API int32_t hl_gather_cold_ahead(hl_ctx* ctx, hl_ubatch* non, const int32_t* d_n_non, const float* host_table,
                                    float* d_cache, int64_t stage_row0, int64_t stage_rows, int32_t* d_cold_rows,
                                    int64_t* d_n_cold, const int32_t* d_prev_cold_rows, const int64_t* d_n_prev,
                                    int32_t* d_fwd_src, void* record_after_index, void* wait_before_move_a,
                                    void* wait_before_move_b, void* stream);

/* The two halves of hl_gather_cold_ahead as separate calls, so that they can go to different streams: hl_index_cold
 * does everything up to and including d_cold_rows, *d_n_cold, d_fwd_src and the unified slots in non->ids (device
 * work only; scratch: the cold region); hl_stage_cold then reads the host rows into the staging window (rows with
 * d_fwd_src[i] >= 0 are left out; d_fwd_src may be NULL).  Issue hl_stage_cold on the stream that also carries the
 * write-backs: stream order then puts the read behind the previous write-back without a stream sitting in an event
 * wait while rows move over the link (on the bench platform a stream blocked in such a wait slowed the write-back
 * running next to it by a factor of five). */
HL_API int32_t hl_index_cold(hl_ctx* ctx, hl_ubatch* non, const int32_t* d_n_non, int64_t stage_row0,
                             int64_t stage_rows, int32_t* d_cold_rows, int64_t* d_n_cold,
                             const int32_t* d_prev_cold_rows, const int64_t* d_n_prev, int32_t* d_fwd_src,
                             void* stream);
/* hl_index_cold in two halves.  hl_index_cold_begin classifies X's lookups and finds the distinct cold rows and the
 * slots: with at most 40 960 cold lookups (20 480 on a device that cannot place a cluster of 16 CTAs) one
 * thread-block cluster does all of it in one kernel; with more, that
 * kernel launches the general search (tile sort, head flags, scan, assignment) from the device, behind itself and
 * ahead of whatever the host queued next -- so the host queues the same two kernels for every mini-batch and never
 * needs to know the count.  The device word hl_index_cold_verdict(ctx) says afterwards which it was: 0 = the cluster
 * kernel, else the number of cold lookups handed on.  hl_index_cold_end does the match against the previous cold rows
 * (general_not_needed is ignored; it dates from when the host queued the general search).  Same arguments as
 * hl_index_cold; both halves on one stream, nothing else of this context's cold-row search between them. */
HL_API int32_t hl_index_cold_begin(hl_ctx* ctx, hl_ubatch* non, const int32_t* d_n_non, int64_t stage_row0,
                                   int64_t stage_rows, int32_t* d_cold_rows, int64_t* d_n_cold, void* stream);
HL_API const int32_t* hl_index_cold_verdict(hl_ctx* ctx);
HL_API int32_t hl_index_cold_end(hl_ctx* ctx, hl_ubatch* non, int64_t stage_row0, int64_t stage_rows,
                                 int32_t* d_cold_rows, int64_t* d_n_cold, const int32_t* d_prev_cold_rows,
                                 const int64_t* d_n_prev, int32_t* d_fwd_src, int32_t general_not_needed, void* stream);
HL_API int32_t hl_stage_cold(hl_ctx* ctx, const float* host_table, float* d_cache, int64_t stage_row0,
                             int64_t stage_rows, const int32_t* d_cold_rows, const int64_t* d_n_cold,
                             const int32_t* d_fwd_src, void* stream);

/* cache[hot_cap + to_stage_row0 + i, :] = cache[hot_cap + from_stage_row0 + d_fwd_src[i], :] for every
 * i < *d_n_cold with d_fwd_src[i] >= 0 (device-to-device; run it after the earlier mini-batch's backward). */
HL_API int32_t hl_forward_cold(hl_ctx* ctx, float* d_cache, int64_t from_stage_row0, int64_t to_stage_row0,
                               int64_t stage_rows, const int32_t* d_fwd_src, const int64_t* d_n_cold, void* stream);

/* hl_scatter_cold from the window [stage_row0, stage_row0 + stage_rows) of the staging area. */
HL_API int32_t hl_scatter_cold_at(hl_ctx* ctx, const float* d_cache, int64_t stage_row0, int64_t stage_rows,
                                  const int32_t* d_cold_rows, const int64_t* d_n_cold, float* host_table,
                                  void* stream);

/* ---------------------------------------------------------------------------------------------------------
 * The pipelined schedule, issued from native code (Section IV: gathering the non-popular working parameters is
 * pipelined with the execution of the popular micro-batch; here the pipeline also spans mini-batches)
 * ------------------------------------------------------------------------------------------------------- */

/* Buffers of one mini-batch in flight; all device memory, caller-owned, sized like the arguments of the calls
 * they are passed to (perm [max_batch]; counts [4]; pop / non as for hl_fragment; cold_rows, fwd_src [window_rows];
 * n_cold [1]; pooled_* [T*max_batch*S, D]; dense_out [max_batch, n_dense] or NULL; sorted_slots / sorted_bags
 * [max_nnz]; sorted_n [4]). */
typedef struct {
    int32_t*  perm;
    int32_t*  counts;
    hl_ubatch pop, non;
    int32_t*  cold_rows;
    int64_t*  n_cold;
    int32_t*  fwd_src;
    float*    pooled_pop;
    float*    pooled_non;
    float*    dense_out;
    int32_t*  sorted_slots;
    int32_t*  sorted_bags;
    int32_t*  sorted_n;
} hl_pipe_set;

typedef struct hl_pipe hl_pipe;

/* A software pipeline over mini-batches on the context `ctx` (which it then uses exclusively): while mini-batch j
 * executes on `main_stream`, the index-only work of mini-batch j + n_sets - 2 (hl_fragment, hl_index_cold,
 * hl_embbag_bwd_prepare2), the host read of j + 1 (hl_stage_cold) and the write-back of j - 1 (hl_scatter_cold_at)
 * run on streams the pipeline creates; rows that consecutive mini-batches share are forwarded between the two
 * staging windows (hl_forward_cold).  The results are those of processing the mini-batches one after the other.
 * d_cache [hot_cap + staging_cap, D] with staging_cap >= 2 * window_rows; host_table as for hl_gather_cold;
 * sets[n_sets] (3 <= n_sets <= 16) are copied.  No device memory is allocated; streams, events and a few pinned host
 * words are.  Returns NULL on invalid arguments or if one of those cannot be created. */
HL_API hl_pipe* hl_pipe_create(hl_ctx* ctx, float* d_cache, float* host_table, int64_t window_rows, int32_t n_sets,
                               const hl_pipe_set* sets, int32_t n_dense, void* main_stream);
/* The same with options (NULL = the defaults, which is what hl_pipe_create uses).  Priorities are CUDA stream
 * priorities: 0 = the default priority, negative = higher, clamped to the device's range.  The main stream is the
 * caller's; to put the bandwidth-bound main work above the ahead-work, create main_stream with a higher priority
 * than the ones given here. */
typedef struct {
    int32_t index_priority;          /* the three streams of index-only ahead-work (fragment, cold-row search, sort) */
    int32_t link_priority;           /* the two streams of host-link transfers (host read, write-back)              */
    int32_t write_back;              /* HL_PIPE_WB_x: when the write-back of mini-batch j runs                       */
} hl_pipe_options;
/* HL_PIPE_WB_OVERLAP (default): as soon as j's backward is over, beside the main work of j + 1.
 * HL_PIPE_WB_EXCLUSIVE: the same, and the main work of j + 1 starts only when it has finished, so that no
 *   bandwidth-bound kernel runs beside a write-back (the index-only ahead-work and the host read still do).
 * HL_PIPE_WB_AFTER_FORWARD: when the popular forward of j + 1 is over (the kernel of the main stream that loses most
 *   next to a write-back); hl_pipe_step then holds j's write-back over until the next hl_pipe_step, or until
 *   hl_pipe_wait_outputs / hl_pipe_drain, whichever comes first (the last step of a run, the one without a next
 *   mini-batch, queues it at once).  The results are the same in all three. */
#define HL_PIPE_WB_OVERLAP       0
#define HL_PIPE_WB_EXCLUSIVE     1
#define HL_PIPE_WB_AFTER_FORWARD 2
HL_API hl_pipe* hl_pipe_create_ex(hl_ctx* ctx, float* d_cache, float* host_table, int64_t window_rows, int32_t n_sets,
                                  const hl_pipe_set* sets, int32_t n_dense, void* main_stream,
                                  const hl_pipe_options* options);
HL_API void hl_pipe_destroy(hl_pipe* p);

/* Order of a mini-batch's main work.  HL_PIPE_ORDER_FIG8 (default): forward O, update O, forward X, update X, as the
 * paper's Fig. 8 draws it.  HL_PIPE_ORDER_EQ5: forward O, forward X, then one update of every touched row with the
 * gradient of the whole mini-batch (Section IV-A, Eq. 5) -- the unfragmented step's result; hl_pipe_step then takes the
 * gradients of O's and X's bags in one array d_grad_pop = [O's bags; X's bags] and ignores d_grad_non.  Set it
 * before the first hl_pipe_submit. */
#define HL_PIPE_ORDER_FIG8 0
#define HL_PIPE_ORDER_EQ5  1
HL_API int32_t hl_pipe_set_order(hl_pipe* p, int32_t order);

/* Queues the ahead-work of the next mini-batch (d_dense may be NULL).  inputs_ready says when its indices, offsets and
 * dense features are complete: NULL = in main_stream's order at the time of the call; a cudaEvent_t = when that event
 * has happened; HL_PIPE_INPUTS_RESIDENT = they already are (the ahead-work then starts without waiting for whatever
 * main_stream still has queued).  Call it n_sets - 2 times before the first hl_pipe_step; afterwards pass the next
 * mini-batch to hl_pipe_step instead.  HL_ECAPACITY if every buffer set is in flight. */
#define HL_PIPE_INPUTS_RESIDENT ((void*)(intptr_t)-1)
HL_API int32_t hl_pipe_submit(hl_pipe* p, const hl_batch* b, const float* d_dense, void* inputs_ready);

/* Queues the main work of the oldest submitted mini-batch: forward and update of O, forward and update of X with the
 * upstream gradients d_grad_pop / d_grad_non ([bags of O, D] / [bags of X, D], in the micro-batches' bag order), and
 * its write-back; and the ahead-work of `next` (may be NULL; next_inputs_ready as for hl_pipe_submit).
 * *set_index = which of the sets holds this mini-batch's perm, counts and pooled vectors; they are complete in
 * main_stream's order, and the set is reused n_sets steps on.  HL_EINVAL if no mini-batch has been submitted,
 * HL_ECAPACITY if `next` finds every buffer set in flight (nothing is queued then).  No call waits for the device. */
HL_API int32_t hl_pipe_step(hl_pipe* p, const float* d_grad_pop, const float* d_grad_non, float lr,
                            const hl_batch* next, const float* d_next_dense, void* next_inputs_ready,
                            int32_t* set_index);

/* Measurement aid: a trace of the pipeline's calls.  Between hl_pipe_trace_begin and hl_pipe_trace_end every library
 * call the pipeline issues whose kind is selected by what_mask (bit HL_SPAN_x) is bracketed by a CUDA event pair on
 * the stream it is issued to, up to max_spans calls (the events are the pipeline's own; they cost a few microseconds
 * of host time per call and no device memory).  Kinds HL_SPAN_KERNEL + HL_TIMER_x bracket single kernels inside those
 * calls: the movers' kernels, the backward's sum kernel, the forward kernel.  hl_pipe_trace_end waits for everything
 * queued (host-side), then writes the recorded spans, in the order they were issued, with times in milliseconds
 * relative to the earliest one; *n_spans = how many.  stream: 0 = main, 1-3 = fragment / sort / cold-row search,
 * 4 = host reads, 5 = write-backs. */
#define HL_SPAN_FRAGMENT     0
#define HL_SPAN_INDEX_BEGIN  1
#define HL_SPAN_INDEX_END    2
#define HL_SPAN_SORT         3
#define HL_SPAN_STAGE        4
#define HL_SPAN_FORWARD_COLD 5
#define HL_SPAN_FWD_POP      6
#define HL_SPAN_BWD_POP      7
#define HL_SPAN_FWD_NON      8
#define HL_SPAN_BWD_NON      9     /* in the order of Eq. 5: the one update of the whole mini-batch */
#define HL_SPAN_SCATTER      10
#define HL_SPAN_KERNEL       16    /* + HL_TIMER_x */
typedef struct {
    int32_t mini_batch;              /* counted from the pipeline's first mini-batch */
    int32_t what;                    /* HL_SPAN_x */
    int32_t stream;
    float   begin_ms, end_ms;
} hl_pipe_span;
HL_API int32_t hl_pipe_trace_begin(hl_pipe* p, int32_t max_spans, uint32_t what_mask);
HL_API int32_t hl_pipe_trace_end(hl_pipe* p, hl_pipe_span* out, int32_t cap, int32_t* n_spans);
/* Makes `stream` wait for the write-back of the last mini-batch stepped (device-side wait). */
HL_API int32_t hl_pipe_wait_outputs(hl_pipe* p, void* stream);
/* Makes `stream` wait until perm and counts of the last mini-batch stepped are final (they are, long before its main
 * work: hl_fragment runs n_sets - 2 mini-batches ahead). */
HL_API int32_t hl_pipe_wait_counts(hl_pipe* p, void* stream);
/* Host waits until everything queued so far has finished. */
HL_API int32_t hl_pipe_drain(hl_pipe* p);

/* ---------------------------------------------------------------------------------------------------------
 * Models with 2^31 rows and more (Section VII-F "Varying Model Size": the synthetic models of 196 to 390 GB), and
 * the hashed lookup of Section V-C: the index-only calls of the path with 64-bit global row ids.
 *
 * Every table still has fewer than 2^31 rows (table-local indices stay int32, the mini-batch layout is unchanged), but
 * the tables together may have more, so popular rows, X's row ids and cold rows are int64.  Nothing is sized by the
 * number of rows: accesses are counted in an open-addressing table of `counter_slots` entries (rounded up to a power
 * of two; it must hold every distinct row the profiled mini-batches touch, HL_ECAPACITY otherwise), and the popular
 * set is an open-addressing table row -> slot of at least 2 * hot_cap_rows entries.  Both are addressed by the
 * randomizer (a 4-round Feistel network on the 32-bit halves of the row id) with linear probing.  Results are those
 * of the dense structures: hl_wide_profile_hot selects by hl_profile_hot's rules (one ranking, count descending, id
 * ascending), popular rows get their slots in ascending id order, hl_wide_fragment and hl_wide_index_cold give
 * hl_fragment's and hl_index_cold's outputs.  The slots they produce feed hl_embbag_fwd / hl_embbag_bwd_* of an
 * ordinary context over the same cache.  Scratch: the caller's workspace (hl_wide_workspace_bytes); the calls of one
 * context must not overlap.
 * ------------------------------------------------------------------------------------------------------- */
typedef struct hl_wide hl_wide;
HL_API size_t hl_wide_workspace_bytes(const hl_geometry* geom, int32_t max_batch, int64_t max_nnz,
                                      int64_t hot_cap_rows, int64_t staging_cap_rows, int64_t counter_slots);
HL_API int32_t hl_wide_create(hl_wide** out, const hl_geometry* geom, int32_t max_batch, int64_t max_nnz,
                              int64_t hot_cap_rows, int64_t staging_cap_rows, int64_t counter_slots,
                              void* d_workspace, size_t ws_bytes);
HL_API int32_t hl_wide_destroy(hl_wide* w);
HL_API int32_t hl_wide_status(hl_wide* w);     /* as hl_status */
/* As hl_profile_hot; d_hot_rows is int64 [hot_cap_rows]; row_bytes is the row payload HL_HOT_BUDGET_BYTES divides by. */
HL_API int32_t hl_wide_profile_hot(hl_wide* w, const hl_batch* b, int32_t reset, int32_t finalize, int32_t policy,
                                   int64_t p_num, int64_t p_den, int32_t row_bytes, int64_t* d_hot_rows,
                                   int64_t* d_n_hot, void* stream);
/* As hl_build_remap without the row load: the hashed remap for d_hot_rows[0 .. *d_n_hot) (strictly ascending). */
HL_API int32_t hl_wide_build_remap(hl_wide* w, const int64_t* d_hot_rows, const int64_t* d_n_hot, void* stream);
/* As hl_fragment (no dense features); X's offsets go to d_non_offsets [T*max_batch*S + 1], its global row ids (int64,
 * -1 for an index outside its table) to d_non_rows [non_cap]. */
HL_API int32_t hl_wide_fragment(hl_wide* w, const hl_batch* b, int32_t* d_perm, int32_t* d_counts, hl_ubatch* pop,
                                int32_t* d_non_offsets, int64_t* d_non_rows, int64_t non_cap, void* stream);
/* As hl_index_cold without windows: d_cold_rows (int64 [staging_cap_rows]) = the distinct non-popular rows of X,
 * ascending; d_non_slots [non_cap] = the unified slot of every lookup of X (hot slot, or hot_cap_rows + rank in
 * d_cold_rows; -1 for a skipped lookup). */
HL_API int32_t hl_wide_index_cold(hl_wide* w, const int32_t* d_non_offsets, const int64_t* d_non_rows, int64_t non_cap,
                                  const int32_t* d_n_non, int32_t* d_non_slots, int64_t* d_cold_rows,
                                  int64_t* d_n_cold, void* stream);

/* No counterpart in the paper: an addition for callers that cannot allocate.
 *
 * Some callers have no way to hand the library a workspace: code that runs where device allocation is forbidden
 * or unavailable (a plug-in inside a host application that owns all device memory and gives none away, a
 * latency-critical loop that must never enter the allocator, a process whose memory budget is already committed).
 * For them this variant of hl_embbag_bwd_sgd needs neither a context nor a workspace: its scratch (sort buffers,
 * histograms, partial sums) is a fixed array of about 3 MB inside the library image, which every GPU that loads
 * the library holds until the process exits.  It calls no cudaMalloc/cudaFree and no allocating routine.
 *
 * Same result as hl_embbag_bwd_sgd: for every distinct id u, cache[u, :] -= lr * sum of d_grad_out[bag(j), :]
 * over the lookups j with ids[j] == u.  d_cache is fp32 [cache_rows, dim]; d_offsets [n_bags + 1] and d_ids [nnz]
 * are a CSR over the bags; d_grad_out is [n_bags, dim]; all device pointers.  n_bags and nnz are given by the
 * host.  d_status (device, may be NULL) receives HL_OK or the first device-side error (HL_EBOUNDS for an id
 * outside the cache; that lookup is skipped).
 *
 * Limits: nnz <= HL_STATIC_MAX_NNZ, n_bags <= HL_STATIC_MAX_NNZ, dim <= HL_STATIC_MAX_DIM; anything larger is
 * refused with HL_ECAPACITY before any work is queued.
 * The first call on a device looks up the device address of the array (cudaGetSymbolAddress, with that device
 * current); make that first call outside any stream capture.
 * All calls on a device share the one array, which still holds the previous call's data: what must start at
 * zero is cleared by the call itself, but two calls that overlap on the GPU (different streams, or different
 * threads) race on it -- serialise them. */
#define HL_STATIC_MAX_NNZ 65536
#define HL_STATIC_MAX_DIM 128
HL_API int32_t hl_embbag_bwd_sgd_static(float* d_cache, int64_t cache_rows, int32_t dim,
                                        const int32_t* d_offsets, const int32_t* d_ids, int32_t n_bags,
                                        int64_t nnz, const float* d_grad_out, float lr, int32_t* d_status,
                                        void* stream);

#ifdef __cplusplus
}
#endif
#endif /* HOTLINE_H_ */
