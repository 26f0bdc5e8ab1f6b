"""Buffer ownership and call order around the C boundary (plumbing only: torch for memory, streams, events).

:class:`Hotline` allocates every buffer the library needs with torch, keeps the context, and issues the calls
of one mini-batch in the order of the paper's pipeline (Fig. 8): fragment, then the cold gather of the
non-popular micro-batch on a side stream while the popular micro-batch runs forward and backward on the main
stream, then the non-popular micro-batch, then the write-back of its cold rows.  No arithmetic happens here.
"""
from __future__ import annotations

from typing import Optional, Sequence

import torch

from . import binding as B


class Hotline:
    def __init__(self, table_rows: Sequence[int], dim: int, bags_per_sample: int, max_batch: int, max_nnz: int,
                 hot_cap_rows: int, staging_cap_rows: int, host_table: torch.Tensor, n_dense: int = 0,
                 device: str = "cuda:0", main_priority: int = 0, side_priority: int = -1):
        """``main_priority`` / ``side_priority``: CUDA stream priorities (0 = default, negative = higher) of the main
        stream and of the streams that carry ahead-work and host-link transfers."""
        if not torch.cuda.is_available():
            raise RuntimeError("the Hotline library needs a CUDA device (there is no CPU fallback)")
        self.device = torch.device(device)
        torch.cuda.set_device(self.device)
        self.table_rows = [int(r) for r in table_rows]
        self.T, self.D, self.S = len(self.table_rows), int(dim), int(bags_per_sample)
        self.N = sum(self.table_rows)
        self.max_batch, self.max_nnz = int(max_batch), int(max_nnz)
        self.hot_cap, self.staging_cap = int(hot_cap_rows), int(staging_cap_rows)
        self.max_bags = self.T * self.max_batch * self.S
        self.n_dense = int(n_dense)
        # host_table: fp32 [N, D], or a list of one fp32 [rows_t, D] tensor per table (a table too large for one
        # allocation).  It must be memory the device can address: from hl_host_alloc (binding.host_table_tensor),
        # pinned host memory, or device memory.  (Not checked here: torch cannot tell for memory it did not allocate.)
        self.host_tables = None
        if isinstance(host_table, (list, tuple)):
            self.host_tables = list(host_table)
            if len(self.host_tables) != self.T or any(
                    t.dtype != torch.float32 or tuple(t.shape) != (r, self.D)
                    for t, r in zip(self.host_tables, self.table_rows)):
                raise ValueError("host_table must be one fp32 [rows_t, D] tensor per table")
            host_table = self.host_tables[0]     # only says "there is a host table" once the per-table bases are set
        elif host_table.dtype != torch.float32 or tuple(host_table.shape) != (self.N, self.D):
            raise ValueError("host_table must be fp32 [N, D]")
        self.host_table = host_table

        dev = self.device
        i32, i64, f32 = torch.int32, torch.int64, torch.float32
        self.geom = B.make_geometry(self.table_rows, self.D, self.S)
        self.ws_bytes = B.hl_workspace_bytes(self.geom, self.max_batch, self.max_nnz, self.hot_cap, self.staging_cap)
        self.workspace = torch.empty(self.ws_bytes, dtype=torch.uint8, device=dev)
        self.cache = torch.zeros((self.hot_cap + self.staging_cap, self.D), dtype=f32, device=dev)
        self.hot_rows = torch.zeros(max(1, self.hot_cap), dtype=i32, device=dev)
        self.n_hot = torch.zeros(1, dtype=i64, device=dev)
        self.perm = torch.zeros(self.max_batch, dtype=i32, device=dev)
        self.counts = torch.zeros(4, dtype=i32, device=dev)          # n_pop, n_non, L_pop, L_non
        self.counts_non = self.counts[1:]                            # view: pointer to n_non
        ids_cap = max(1, self.max_nnz)
        self.pop_offsets = torch.zeros(self.max_bags + 1, dtype=i32, device=dev)
        self.pop_ids = torch.zeros(ids_cap, dtype=i32, device=dev)
        self.non_offsets = torch.zeros(self.max_bags + 1, dtype=i32, device=dev)
        self.non_ids = torch.zeros(ids_cap, dtype=i32, device=dev)
        self.pop = B.make_ubatch(self.pop_offsets, self.pop_ids, self.max_nnz)
        self.non = B.make_ubatch(self.non_offsets, self.non_ids, self.max_nnz)
        self.cold_rows = torch.zeros(max(1, self.staging_cap), dtype=i32, device=dev)
        self.n_cold = torch.zeros(1, dtype=i64, device=dev)
        self.pooled_pop = torch.zeros((self.max_bags, self.D), dtype=f32, device=dev)
        self.pooled_non = torch.zeros((self.max_bags, self.D), dtype=f32, device=dev)
        self.dense_out = torch.zeros((self.max_batch, self.n_dense), dtype=f32, device=dev) if n_dense else None
        self.main_priority, self.side_priority = int(main_priority), int(side_priority)
        self.main = torch.cuda.Stream(device=dev, priority=self.main_priority)
        self.side = torch.cuda.Stream(device=dev, priority=self.side_priority)
        self.ev_frag = torch.cuda.Event()
        self.ev_gather = torch.cuda.Event()
        self.ev_pop_done = torch.cuda.Event()
        self.ctx = B.hl_create(self.geom, self.max_batch, self.max_nnz, self.hot_cap, self.staging_cap,
                               self.workspace, self.ws_bytes)
        if self.host_tables is not None:
            B.hl_set_host_tables(self.ctx, self.host_tables)

    # ---- life cycle ------------------------------------------------------------------------------------------
    def close(self) -> None:
        if getattr(self, "ctx", None):
            torch.cuda.synchronize(self.device)
            B.hl_destroy(self.ctx)
            self.ctx = None

    def __enter__(self):
        return self

    def __exit__(self, *exc):
        self.close()

    def __del__(self):  # pragma: no cover
        try:
            self.close()
        except Exception:
            pass

    def status(self, raise_on_error: bool = True) -> int:
        return B.hl_status(self.ctx, raise_on_error)

    def _batch(self, indices: torch.Tensor, offsets: torch.Tensor, batch: int) -> B.hl_batch:
        assert indices.dtype == torch.int32 and offsets.dtype == torch.int32 and indices.is_cuda and offsets.is_cuda
        assert offsets.numel() == self.T * batch * self.S + 1
        return B.make_batch(indices, offsets, batch, indices.numel())

    # ---- learning phase --------------------------------------------------------------------------------------
    def profile(self, indices: Optional[torch.Tensor], offsets: Optional[torch.Tensor], batch: int = 0,
                reset: bool = False, finalize: bool = False, policy: int = B.HL_HOT_TOPK_ROWS, p_num: int = 0,
                p_den: int = 1) -> None:
        b = self._batch(indices, offsets, batch) if indices is not None else None
        B.hl_profile_hot(self.ctx, b, reset, finalize, policy, p_num, p_den, self.hot_rows, self.n_hot,
                         self.main.cuda_stream)

    def tracker_init(self, n_sets: int, ways: int = 16) -> None:
        """The approximate access logger (SRRIP table of n_sets x ways row tags) instead of the exact counters:
        tracker_init, tracker_update per sampled mini-batch, then tracker_select."""
        self.trk_shape = (int(n_sets), int(ways))
        self.trk_tags = torch.empty(n_sets * ways, dtype=torch.int32, device=self.device)
        self.trk_rrpv = torch.empty(n_sets * ways, dtype=torch.uint8, device=self.device)
        self.trk_hits = torch.zeros(1, dtype=torch.int64, device=self.device)
        B.hl_tracker_reset(self.ctx, self.trk_tags, self.trk_rrpv, n_sets, ways, self.trk_hits,
                           self.main.cuda_stream)

    def tracker_update(self, indices: torch.Tensor, offsets: torch.Tensor, batch: int) -> None:
        n_sets, ways = self.trk_shape
        B.hl_tracker_update(self.ctx, self._batch(indices, offsets, batch), self.trk_tags, self.trk_rrpv, n_sets,
                            ways, self.trk_hits, self.main.cuda_stream)

    def tracker_select(self, policy: int = B.HL_HOT_TOPK_ROWS, p_num: int = 0, p_den: int = 1) -> None:
        """The popular set = the rows the logger holds, clipped by the policy (most recently re-referenced first)."""
        n_sets, ways = self.trk_shape
        B.hl_tracker_export(self.ctx, self.trk_tags, self.trk_rrpv, n_sets, ways, self.main.cuda_stream)
        B.hl_profile_hot(self.ctx, None, False, True, policy, p_num, p_den, self.hot_rows, self.n_hot,
                         self.main.cuda_stream)

    def set_hot_rows(self, rows: torch.Tensor) -> None:
        """Installs a caller-chosen popular set (ascending global ids) instead of a profiled one."""
        n = rows.numel()
        assert n <= self.hot_cap
        with torch.cuda.stream(self.main):
            self.hot_rows[:n].copy_(rows.to(torch.int32), non_blocking=True)
            self.n_hot.fill_(n)

    def build_remap(self, load_rows: bool = True, remap_out: Optional[torch.Tensor] = None) -> None:
        B.hl_build_remap(self.ctx, self.hot_rows, self.n_hot, self.host_table if load_rows else None, self.cache,
                         remap_out, self.main.cuda_stream)

    def flush_hot(self) -> None:
        """Writes the popular rows' current values back to the host table (do this before re-learning the set)."""
        B.hl_flush_hot(self.ctx, self.cache, self.hot_rows, self.n_hot, self.host_table, self.main.cuda_stream)

    # ---- acceleration phase: single calls ---------------------------------------------------------------------
    def fragment(self, indices, offsets, batch: int, dense: Optional[torch.Tensor] = None) -> None:
        B.hl_fragment(self.ctx, self._batch(indices, offsets, batch), dense, self.n_dense if dense is not None else 0,
                      self.perm, self.counts, self.pop, self.non, self.dense_out if dense is not None else None,
                      self.main.cuda_stream)

    def gather_cold(self, stream: Optional[torch.cuda.Stream] = None) -> None:
        s = stream or self.main
        B.hl_gather_cold(self.ctx, self.non, self.counts_non, self.host_table, self.cache, self.cold_rows,
                         self.n_cold, s.cuda_stream)

    def fwd_pop(self) -> None:
        B.hl_embbag_fwd(self.ctx, self.cache, self.pop, self.counts, self.pooled_pop, self.main.cuda_stream)

    def fwd_non(self) -> None:
        B.hl_embbag_fwd(self.ctx, self.cache, self.non, self.counts_non, self.pooled_non, self.main.cuda_stream)

    def bwd_pop(self, grad: torch.Tensor, lr: float) -> None:
        B.hl_embbag_bwd_sgd(self.ctx, self.cache, self.pop, self.counts, grad, lr, self.main.cuda_stream)

    def bwd_non(self, grad: torch.Tensor, lr: float) -> None:
        B.hl_embbag_bwd_sgd(self.ctx, self.cache, self.non, self.counts_non, grad, lr, self.main.cuda_stream)

    def scatter_cold(self) -> None:
        B.hl_scatter_cold(self.ctx, self.cache, self.cold_rows, self.n_cold, self.host_table, self.main.cuda_stream)

    # ---- acceleration phase: one mini-batch --------------------------------------------------------------------
    def step(self, indices, offsets, batch: int, grad_pop: torch.Tensor, grad_non: torch.Tensor, lr: float,
             dense: Optional[torch.Tensor] = None, deferred: bool = False, overlap: bool = True,
             timers: Optional[dict] = None) -> None:
        """One mini-batch through the pipeline.  ``grad_pop`` / ``grad_non`` are the upstream gradients of the
        pooled outputs of O and X (rows in the micro-batches' own bag order).  ``deferred`` runs both forwards
        before both backwards; ``overlap=False`` keeps the cold gather on the main stream.  ``timers``: a dict
        that receives, per call name, a list of (start, end) CUDA events recorded on the stream of that call."""

        def timed(name, stream, fn):
            if timers is None or ("only" in timers and name not in timers["only"]):
                fn()
                return
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(stream)
            fn()
            b.record(stream)
            timers.setdefault(name, []).append((a, b))

        m = self.main
        timed("fragment", m, lambda: self.fragment(indices, offsets, batch, dense))
        if overlap:
            self.ev_frag.record(m)
            self.side.wait_event(self.ev_frag)
            timed("gather_cold", self.side, lambda: self.gather_cold(self.side))
            self.ev_gather.record(self.side)
        else:
            timed("gather_cold", m, lambda: self.gather_cold(m))
        timed("fwd_pop", m, self.fwd_pop)
        if not deferred:
            timed("bwd_pop", m, lambda: self.bwd_pop(grad_pop, lr))
        if overlap:
            m.wait_event(self.ev_gather)
        timed("fwd_non", m, self.fwd_non)
        if deferred:
            timed("bwd_pop", m, lambda: self.bwd_pop(grad_pop, lr))
        timed("bwd_non", m, lambda: self.bwd_non(grad_non, lr))
        timed("scatter_cold", m, self.scatter_cold)

    def synchronize(self) -> None:
        self.main.synchronize()
        self.side.synchronize()


class _BatchSet:
    """Index buffers and outputs of one mini-batch in flight."""

    def __init__(self, h: "Hotline"):
        dev, i32, i64, f32 = h.device, torch.int32, torch.int64, torch.float32
        ids_cap = max(1, h.max_nnz)
        self.perm = torch.zeros(h.max_batch, dtype=i32, device=dev)
        self.counts = torch.zeros(4, dtype=i32, device=dev)
        self.counts_non = self.counts[1:]
        self.pop_offsets = torch.zeros(h.max_bags + 1, dtype=i32, device=dev)
        self.pop_ids = torch.zeros(ids_cap, dtype=i32, device=dev)
        self.non_offsets = torch.zeros(h.max_bags + 1, dtype=i32, device=dev)
        self.non_ids = torch.zeros(ids_cap, dtype=i32, device=dev)
        self.pop = B.make_ubatch(self.pop_offsets, self.pop_ids, h.max_nnz)
        self.non = B.make_ubatch(self.non_offsets, self.non_ids, h.max_nnz)
        self.cold_rows = torch.zeros(max(1, h.window_rows), dtype=i32, device=dev)
        self.n_cold = torch.zeros(1, dtype=i64, device=dev)
        self.fwd_src = torch.full((max(1, h.window_rows),), -1, dtype=i32, device=dev)
        self.pooled_pop = torch.zeros((h.max_bags, h.D), dtype=f32, device=dev)
        self.pooled_non = torch.zeros((h.max_bags, h.D), dtype=f32, device=dev)
        self.dense_out = torch.zeros((h.max_batch, h.n_dense), dtype=f32, device=dev) if h.n_dense else None
        # events whose handles the library records or waits on: record each once so that the handle exists
        self.ev_index = torch.cuda.Event()
        self.ev_gather = torch.cuda.Event()
        self.ev_forward = torch.cuda.Event()
        self.ev_x = torch.cuda.Event()
        self.ev_scatter = torch.cuda.Event()
        self.ev_inputs = torch.cuda.Event()
        self.ev_frag = torch.cuda.Event()
        self.ev_prep_pop = torch.cuda.Event()
        self.ev_prep_non = torch.cuda.Event()
        for e in (self.ev_index, self.ev_gather, self.ev_forward, self.ev_x, self.ev_scatter, self.ev_inputs,
                  self.ev_frag, self.ev_prep_pop, self.ev_prep_non):
            e.record(h.main)
        # (slot, bag) pairs of both micro-batches sorted by slot, prepared ahead of the backward passes
        self.sorted_pop = (torch.zeros(ids_cap, dtype=i32, device=dev), torch.zeros(ids_cap, dtype=i32, device=dev),
                           torch.zeros(1, dtype=i32, device=dev))
        self.sorted_non = (torch.zeros(ids_cap, dtype=i32, device=dev), torch.zeros(ids_cap, dtype=i32, device=dev),
                           torch.zeros(1, dtype=i32, device=dev))
        # the pairs of O and X sorted together (O's block first); [2] = lookups of O, of X, and their sum
        self.sorted_all = (torch.zeros(ids_cap, dtype=i32, device=dev), torch.zeros(ids_cap, dtype=i32, device=dev),
                           torch.zeros(4, dtype=i32, device=dev))


class PipelinedHotline(Hotline):
    """The same path, software-pipelined across mini-batches, issued from Python (NativePipelinedHotline issues the
    default variant from C).  While mini-batch j executes on the main stream, the index-only work of mini-batch
    j+lookahead (fragment, cold-row search, backward sort) runs on three side streams, the host rows of j+1 are read on
    a link stream, and j-1's cold rows are written back on another.  The result is that of processing the mini-batches
    one after the other: a cold row that j+1 shares with j is not read from the host but copied from j's staging
    window after j's backward (hl_forward_cold), and the host rows of j+1 are read only after j-1's write-back has
    finished.

    lookahead + 2 sets of index buffers rotate over the mini-batches, two windows of the staging area alternate.

    ``overlap_link=True`` (default): the read of j+1's host rows starts as soon as j-1's write-back is done and
    overlaps j's execution and write-back, with the rows j+1 shares with j forwarded between the staging windows.
    ``overlap_link=False``: the host rows of j+1 are read after j's write-back has finished, so the two transfers
    follow each other on the link and no forwarding is needed; fragment and the search for the distinct cold rows of
    j+1 still run under j's execution.  (Which is faster depends on the host table's memory: with large-page
    device mappings (hl_host_alloc) 0.30 against 0.43 ms per DLRM-large-like mini-batch; with 4 KB mappings
    (cudaHostAlloc) reads and write-backs compete for address translations and it was the other way round, 0.84
    against 0.65 ms.)

        p.start(idx0, off0, B, dense0, more=[(idx1, off1, B, dense1)])      # ahead-work of `lookahead` mini-batches
        for j in range(n):
            s = p.step(grad_pop, grad_non, lr, next_batch=(idx, off, B, dense) or None)   # the next one not yet given
            ... p.sets[s].pooled_pop / pooled_non are mini-batch j's outputs once the main stream gets there
        p.drain()
    """

    def __init__(self, table_rows, dim, bags_per_sample, max_batch, max_nnz, hot_cap_rows, window_rows, host_table,
                 n_dense: int = 0, device: str = "cuda:0", overlap_link: bool = True, sort_ahead: bool = True,
                 combined_sort: bool = True, lookahead: int = 2, main_priority: int = 0, side_priority: int = -1):
        self.overlap_link = bool(overlap_link)
        # sort_ahead (with overlap_link): the sorts of the two backward passes, which depend on the ids only, are
        # part of the ahead-work (hl_embbag_bwd_prepare on a side stream); the main stream keeps the forwards and
        # the gradient sums + updates (hl_embbag_bwd_apply)
        self.sort_ahead = bool(sort_ahead) and self.overlap_link
        # combined_sort (with sort_ahead): one sort over the pairs of O and X (hl_embbag_bwd_prepare2) instead of two
        self.combined_sort = bool(combined_sort) and self.sort_ahead
        # lookahead (with sort_ahead): the index-only part of the ahead-work (fragment, cold-row search, sort) runs
        # this many mini-batches ahead of the main stream; the read of the host rows stays one mini-batch ahead, but
        # no longer has that index work in front of it.  start() takes lookahead mini-batches, step() the one
        # lookahead places after the mini-batch it executes.
        self.lookahead = max(1, int(lookahead)) if self.sort_ahead else 1
        self.window_rows = int(window_rows)
        super().__init__(table_rows, dim, bags_per_sample, max_batch, max_nnz, hot_cap_rows, 2 * self.window_rows,
                         host_table, n_dense=n_dense, device=device, main_priority=main_priority,
                         side_priority=side_priority)
        self.n_sets = self.lookahead + 2
        self.sets = [_BatchSet(self) for _ in range(self.n_sets)]
        self.sides = [self.side] + [torch.cuda.Stream(device=self.device, priority=self.side_priority)
                                    for _ in range(2)]
        self.wb = torch.cuda.Stream(device=self.device, priority=self.side_priority)
        self.link = torch.cuda.Stream(device=self.device, priority=self.side_priority)
        self.j_submitted = 0      # mini-batches whose ahead-work (host read included) has been issued
        self.j_indexed = 0        # sort_ahead schedule: mini-batches whose index-only ahead-work has been issued
        self.j_done = 0           # mini-batches whose main work has been issued
        torch.cuda.synchronize(self.device)

    @staticmethod
    def _timed(timers, name, stream, fn):
        if timers is None or ("only" in timers and name not in timers["only"]):
            fn()
            return
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(stream)
        fn()
        b.record(stream)
        timers.setdefault(name, []).append((a, b))

    def _submit_index(self, indices, offsets, batch: int, dense=None, timers=None) -> None:
        """Index-only ahead-work of the next mini-batch in the sort_ahead schedule.  Stream A: fragment.  Stream C:
        cold-row search (after fragment).  Stream B: the backward sorts (after the cold-row search, or O's after
        fragment).  Three streams, so that the three chains of small kernels of successive mini-batches overlap."""
        j, n = self.j_indexed, self.n_sets
        st, sa, sb, sc = self.sets[j % n], self.sides[0], self.sides[1], self.sides[2]
        prev = self.sets[(j - 1) % n] if j >= 1 else None
        w = (j % 2) * self.window_rows
        sa.wait_event(st.ev_inputs)
        if j >= n:
            sa.wait_event(st.ev_scatter)                 # the buffers of this set were mini-batch j-n_sets's
        self._timed(timers, "fragment", sa, lambda: B.hl_fragment(
            self.ctx, self._batch(indices, offsets, batch), dense, self.n_dense if dense is not None else 0,
            st.perm, st.counts, st.pop, st.non, st.dense_out if dense is not None else None, sa.cuda_stream))
        st.ev_frag.record(sa)
        sc.wait_event(st.ev_frag)
        if j >= n:
            sc.wait_event(st.ev_scatter)
        self._timed(timers, "index_cold", sc, lambda: B.hl_index_cold(
            self.ctx, st.non, st.counts_non, w, self.window_rows, st.cold_rows, st.n_cold,
            prev.cold_rows if prev is not None else None, prev.n_cold if prev is not None else None, st.fwd_src,
            sc.cuda_stream))
        st.ev_index.record(sc)
        if self.combined_sort:
            sb.wait_event(st.ev_index)
            self._timed(timers, "sort_all", sb, lambda: B.hl_embbag_bwd_prepare2(
                self.ctx, st.pop, st.counts, st.non, st.counts_non, st.sorted_all[0], st.sorted_all[1],
                st.sorted_all[2], sb.cuda_stream))
            st.ev_prep_pop.record(sb)
            st.ev_prep_non.record(sb)
        else:
            sb.wait_event(st.ev_frag)
            self._timed(timers, "sort_pop", sb, lambda: B.hl_embbag_bwd_prepare(
                self.ctx, st.pop, st.counts, st.sorted_pop[0], st.sorted_pop[1], st.sorted_pop[2], sb.cuda_stream))
            st.ev_prep_pop.record(sb)
            sb.wait_event(st.ev_index)
            self._timed(timers, "sort_non", sb, lambda: B.hl_embbag_bwd_prepare(
                self.ctx, st.non, st.counts_non, st.sorted_non[0], st.sorted_non[1], st.sorted_non[2],
                sb.cuda_stream))
            st.ev_prep_non.record(sb)
        self.j_indexed += 1

    def _submit_link(self, timers=None) -> None:
        """The host read of the oldest indexed mini-batch whose rows are not staged yet (link stream)."""
        j, n = self.j_submitted, self.n_sets
        assert j < self.j_indexed
        st, lk = self.sets[j % n], self.link
        prev = self.sets[(j - 1) % n] if j >= 1 else None
        w = (j % 2) * self.window_rows
        lk.wait_event(st.ev_index)
        if j >= 2:
            lk.wait_event(self.sets[(j - 2) % n].ev_scatter)    # host rows of j-2 are final; its window is free
        if prev is not None:
            lk.wait_event(prev.ev_forward)                       # j-1 took what it needs out of this window
        self._timed(timers, "gather_cold", lk, lambda: B.hl_stage_cold(
            self.ctx, self.host_table, self.cache, w, self.window_rows, st.cold_rows, st.n_cold,
            st.fwd_src if prev is not None else None, lk.cuda_stream))
        st.ev_gather.record(lk)
        self.j_submitted += 1

    def _step_sorted(self, grad_pop, grad_non, lr, next_batch, timers) -> int:
        j, n = self.j_done, self.n_sets
        st, m = self.sets[j % n], self.main
        s_main = m.cuda_stream
        w0, w1 = (j % 2) * self.window_rows, ((j + 1) % 2) * self.window_rows
        if next_batch is not None:
            self.sets[self.j_indexed % n].ev_inputs.record(m)
        m.wait_event(st.ev_index)
        # rows shared with mini-batch j-1 come out of its staging window once its backward is done; on the link
        # stream, between the host reads of j and of j+1, so that O's work on the main stream does not wait for it
        lk = self.link
        if j >= 1:
            lk.wait_event(st.ev_index)
            lk.wait_event(self.sets[(j - 1) % n].ev_x)
            B.hl_forward_cold(self.ctx, self.cache, w1, w0, self.window_rows, st.fwd_src, st.n_cold, lk.cuda_stream)
        st.ev_forward.record(lk)
        if self.j_submitted < self.j_indexed:
            self._submit_link(timers)                    # mini-batch j+1, indexed during an earlier step
        if next_batch is not None:
            self._submit_index(*next_batch, timers=timers)
            if self.j_submitted == j + 1:
                self._submit_link(timers)                # lookahead 1: j+1 was indexed only just now
        t = lambda name, stream, fn: self._timed(timers, name, stream, fn)   # noqa: E731
        t("fwd_pop", m, lambda: B.hl_embbag_fwd(self.ctx, self.cache, st.pop, st.counts, st.pooled_pop, s_main))
        m.wait_event(st.ev_prep_pop)
        if self.combined_sort:
            sa_ = st.sorted_all
            t("bwd_pop", m, lambda: B.hl_embbag_bwd_apply2(self.ctx, self.cache, sa_[0], sa_[1], sa_[2], 0, grad_pop,
                                                           lr, s_main))
        else:
            t("bwd_pop", m, lambda: B.hl_embbag_bwd_apply(self.ctx, self.cache, st.sorted_pop[0], st.sorted_pop[1],
                                                          st.sorted_pop[2], grad_pop, lr, s_main))
        m.wait_event(st.ev_gather)
        m.wait_event(st.ev_forward)
        t("fwd_non", m, lambda: B.hl_embbag_fwd(self.ctx, self.cache, st.non, st.counts_non, st.pooled_non, s_main))
        m.wait_event(st.ev_prep_non)
        if self.combined_sort:
            t("bwd_non", m, lambda: B.hl_embbag_bwd_apply2(self.ctx, self.cache, sa_[0], sa_[1], sa_[2], 1, grad_non,
                                                           lr, s_main))
        else:
            t("bwd_non", m, lambda: B.hl_embbag_bwd_apply(self.ctx, self.cache, st.sorted_non[0], st.sorted_non[1],
                                                          st.sorted_non[2], grad_non, lr, s_main))
        st.ev_x.record(m)
        self.wb.wait_event(st.ev_x)
        t("scatter_cold", self.wb, lambda: B.hl_scatter_cold_at(
            self.ctx, self.cache, w0, self.window_rows, st.cold_rows, st.n_cold, self.host_table,
            self.wb.cuda_stream))
        st.ev_scatter.record(self.wb)
        self.j_done += 1
        return j % n

    def _submit(self, indices, offsets, batch: int, dense=None, timers=None) -> None:
        if self.sort_ahead:
            self._submit_index(indices, offsets, batch, dense, timers)
            if self.j_submitted == self.j_done:
                self._submit_link(timers)
            return
        j = self.j_submitted
        st, side = self.sets[j % 3], self.sides[j % 2]
        side.wait_event(st.ev_inputs)                    # the caller prepared the inputs on the main stream
        if j >= 3:
            side.wait_event(st.ev_scatter)               # set j%3 was mini-batch j-3's: long done, stated anyway
        prev = self.sets[(j - 1) % 3] if j >= 1 else None
        if prev is not None:
            side.wait_event(prev.ev_index)               # its cold set is final; fragment/cold scratch is free
        if self.overlap_link:
            excl = prev
            wait_a = self.sets[(j - 2) % 3].ev_scatter if j >= 2 else None   # host rows of j-2 are final
            wait_b = prev.ev_forward if prev is not None else None           # j-1 took what it needs from the window
        else:
            excl = None
            wait_a = wait_b = None
            if j >= 2:
                # keep this mini-batch's fragment / index kernels away from the write-back of mini-batch j-2: they
                # then run next to the read of j-1's host rows instead
                side.wait_event(self.sets[(j - 2) % 3].ev_scatter)
        self._timed(timers, "fragment", side, lambda: B.hl_fragment(
            self.ctx, self._batch(indices, offsets, batch), dense, self.n_dense if dense is not None else 0,
            st.perm, st.counts, st.pop, st.non, st.dense_out if dense is not None else None, side.cuda_stream))
        if self.overlap_link:
            self._timed(timers, "gather_cold", side, lambda: B.hl_gather_cold_ahead(
                self.ctx, st.non, st.counts_non, self.host_table, self.cache, (j % 2) * self.window_rows,
                self.window_rows, st.cold_rows, st.n_cold,
                excl.cold_rows if excl is not None else None, excl.n_cold if excl is not None else None, st.fwd_src,
                st.ev_index, wait_a, wait_b, side.cuda_stream))
            st.ev_gather.record(side)
        else:
            # index work on the side stream; the read of the host rows on the write-back stream, behind the
            # write-back of the mini-batch before (stream order, no stream parked in an event wait meanwhile)
            self._timed(timers, "index_cold", side, lambda: B.hl_index_cold(
                self.ctx, st.non, st.counts_non, (j % 2) * self.window_rows, self.window_rows, st.cold_rows,
                st.n_cold, None, None, None, side.cuda_stream))
            st.ev_index.record(side)
            self.wb.wait_event(st.ev_index)
            self._timed(timers, "gather_cold", self.wb, lambda: B.hl_stage_cold(
                self.ctx, self.host_table, self.cache, (j % 2) * self.window_rows, self.window_rows, st.cold_rows,
                st.n_cold, None, self.wb.cuda_stream))
            st.ev_gather.record(self.wb)
        self.j_submitted += 1

    def start(self, indices, offsets, batch: int, dense=None, more=(), inputs_ready=None) -> None:
        """Ahead-work of the first mini-batch; ``more`` = the (indices, offsets, batch, dense) tuples of the
        lookahead - 1 mini-batches after it (fewer if the run is shorter).  (``inputs_ready`` is accepted for the
        interface it shares with NativePipelinedHotline; this scheduler always orders the ahead-work after the main
        stream.)"""
        assert self.j_submitted == self.j_done, "start() only with nothing in flight"
        assert len(more) <= self.lookahead - 1
        if self.sort_ahead:
            self.j_indexed = self.j_submitted
        for nb in [(indices, offsets, batch, dense)] + [tuple(x) for x in more]:
            k = self.j_indexed if self.sort_ahead else self.j_submitted
            self.sets[k % self.n_sets].ev_inputs.record(self.main)
            self._submit(*nb)

    def step(self, grad_pop: torch.Tensor, grad_non: torch.Tensor, lr: float, next_batch=None, timers=None,
             inputs_ready=None) -> int:
        """Main work of the oldest submitted mini-batch; ``next_batch`` = (indices, offsets, batch, dense) of
        the mini-batch ``lookahead`` places after it (its ahead-work is issued here), or None at the end.  Returns
        the index of the buffer set that holds this mini-batch's outputs."""
        j = self.j_done
        assert self.j_submitted >= j + 1, "call start() first"
        if self.sort_ahead:
            return self._step_sorted(grad_pop, grad_non, lr, next_batch, timers)
        st, m = self.sets[j % 3], self.main
        s_main = m.cuda_stream
        w0, w1 = (j % 2) * self.window_rows, ((j + 1) % 2) * self.window_rows
        if next_batch is not None:
            self.sets[(j + 1) % 3].ev_inputs.record(m)   # the next mini-batch's inputs are ready at this point
        m.wait_event(st.ev_index)
        if not self.overlap_link and j >= 1:
            # The write-back of mini-batch j-1 gets the chip to itself; this mini-batch's popular work starts when it
            # is done, next to the read of its own cold rows.  (This mattered with a host table in cudaHostAlloc
            # memory, whose 4 KB device mappings made a write-back next to other kernels 5 times slower; with a table
            # from hl_host_alloc it costs about 3 %.)
            m.wait_event(self.sets[(j - 1) % 3].ev_scatter)
        if self.overlap_link and j >= 1:
            # rows shared with mini-batch j-1 come from its staging window (its backward ran on this stream)
            B.hl_forward_cold(self.ctx, self.cache, w1, w0, self.window_rows, st.fwd_src, st.n_cold, s_main)
        st.ev_forward.record(m)
        if next_batch is not None and self.overlap_link:
            self._submit(*next_batch, timers=timers)
        t = lambda name, stream, fn: self._timed(timers, name, stream, fn)   # noqa: E731
        t("fwd_pop", m, lambda: B.hl_embbag_fwd(self.ctx, self.cache, st.pop, st.counts, st.pooled_pop, s_main))
        t("bwd_pop", m, lambda: B.hl_embbag_bwd_sgd(self.ctx, self.cache, st.pop, st.counts, grad_pop, lr, s_main))
        m.wait_event(st.ev_gather)
        t("fwd_non", m, lambda: B.hl_embbag_fwd(self.ctx, self.cache, st.non, st.counts_non, st.pooled_non, s_main))
        t("bwd_non", m, lambda: B.hl_embbag_bwd_sgd(self.ctx, self.cache, st.non, st.counts_non, grad_non, lr,
                                                    s_main))
        st.ev_x.record(m)
        self.wb.wait_event(st.ev_x)
        t("scatter_cold", self.wb, lambda: B.hl_scatter_cold_at(
            self.ctx, self.cache, w0, self.window_rows, st.cold_rows, st.n_cold, self.host_table,
            self.wb.cuda_stream))
        st.ev_scatter.record(self.wb)
        if next_batch is not None and not self.overlap_link:
            self._submit(*next_batch, timers=timers)     # its host rows are read after the write-back just queued
        self.j_done += 1
        return j % 3

    @property
    def idle(self) -> bool:
        return self.j_submitted == self.j_done

    def wait_outputs(self) -> None:
        """The main stream waits for the last write-back (device-side)."""
        self.main.wait_stream(self.wb)

    def wait_counts(self, stream: torch.cuda.Stream) -> None:
        """``stream`` waits until perm and counts of the mini-batch last stepped are final."""
        if self.j_done >= 1:
            stream.wait_event(self.sets[(self.j_done - 1) % self.n_sets].ev_index)

    def drain(self) -> None:
        """Waits until everything issued so far, write-backs included, has finished."""
        for s in [self.main, self.wb, self.link] + self.sides:
            s.synchronize()


class NativePipelinedHotline(Hotline):
    """The default schedule of :class:`PipelinedHotline` (index work ``lookahead`` mini-batches ahead on three
    streams, one combined backward sort, host reads overlapping write-backs, shared rows forwarded), issued by the
    library itself (hl_pipe_*): one C call per mini-batch instead of some sixty Python-level calls, which is what
    bounds small mini-batches.  Same results, same buffers (``sets``), same call pattern:

        p.start(idx0, off0, B, dense0, more=[(idx1, off1, B, dense1)])    # lookahead mini-batches
        for j in range(n):
            s = p.step(grad_pop, grad_non, lr, next_batch=(idx, off, B, dense) or None)
        p.drain()
    """

    def __init__(self, table_rows, dim, bags_per_sample, max_batch, max_nnz, hot_cap_rows, window_rows, host_table,
                 n_dense: int = 0, device: str = "cuda:0", lookahead: int = 2, order: str = "fig8",
                 main_priority: int = -1, index_priority: int = 0, link_priority: int = 0, mover_ctas: int = 0,
                 scatter_ctas: int = 0, write_back: str = "overlap"):
        """``order``: "fig8" = forward O, update O, forward X, update X (the paper's Fig. 8); "eq5" = both forwards,
        then one update of every touched row with the whole mini-batch's gradient (Eq. 5; the unfragmented step's
        result): step() then takes ``grad_pop`` = [gradients of O's bags; gradients of X's bags] and no ``grad_non``.
        ``main_priority`` / ``index_priority`` / ``link_priority``: CUDA stream priorities (0 = default, negative =
        higher) of the main stream (bandwidth-bound forwards and updates), of the index-only ahead-work and of the
        host-link transfers.  ``mover_ctas`` / ``scatter_ctas``: hl_set_mover_ctas (0 = the library's default).
        ``write_back``: when a mini-batch's write-back runs: "overlap" = right after its backward, beside the next
        mini-batch's main work; "exclusive" = the same, and the next mini-batch's main work waits for it;
        "after_forward" = when the next mini-batch's popular forward is over."""
        assert order in ("fig8", "eq5")
        wb_modes = {"overlap": B.HL_PIPE_WB_OVERLAP, "exclusive": B.HL_PIPE_WB_EXCLUSIVE,
                    "after_forward": B.HL_PIPE_WB_AFTER_FORWARD}
        assert write_back in wb_modes
        self.order = order
        self.window_rows = int(window_rows)
        self.lookahead = max(1, int(lookahead))
        super().__init__(table_rows, dim, bags_per_sample, max_batch, max_nnz, hot_cap_rows, 2 * self.window_rows,
                         host_table, n_dense=n_dense, device=device, main_priority=main_priority,
                         side_priority=index_priority)
        self.n_sets = self.lookahead + 2
        self.sets = [_BatchSet(self) for _ in range(self.n_sets)]
        c_sets = []
        for st in self.sets:
            c_sets.append(B.hl_pipe_set(
                B._ptr(st.perm), B._ptr(st.counts), st.pop, st.non, B._ptr(st.cold_rows), B._ptr(st.n_cold),
                B._ptr(st.fwd_src), B._ptr(st.pooled_pop), B._ptr(st.pooled_non), B._ptr(st.dense_out),
                B._ptr(st.sorted_all[0]), B._ptr(st.sorted_all[1]), B._ptr(st.sorted_all[2])))
        torch.cuda.synchronize(self.device)
        if mover_ctas or scatter_ctas:
            B.hl_set_mover_ctas(self.ctx, mover_ctas, scatter_ctas)
        self.pipe = B.hl_pipe_create_ex(self.ctx, self.cache, self.host_table, self.window_rows, c_sets, self.n_dense,
                                        self.main.cuda_stream, index_priority=index_priority,
                                        link_priority=link_priority, write_back=wb_modes[write_back])
        if order == "eq5":
            B.hl_pipe_set_order(self.pipe, B.HL_PIPE_ORDER_EQ5)
        self.in_flight = 0
        self.j_done = 0           # mini-batches stepped so far (mini-batch j stages its cold rows in window j % 2)

    def trace_begin(self, max_spans: int, what_mask: int = B.HL_SPAN_ALL) -> None:
        """Records a CUDA event pair around the library calls (and the timed kernels inside them) that the
        following steps issue; trace_end() drains the pipeline and returns the spans."""
        self._trace_cap = int(max_spans)
        B.hl_pipe_trace_begin(self.pipe, max_spans, what_mask)

    def trace_end(self):
        return B.hl_pipe_trace_end(self.pipe, self._trace_cap)

    def _hl_batch(self, nb):
        indices, offsets, batch, dense = nb
        return self._batch(indices, offsets, batch), (dense if self.n_dense else None)

    def start(self, indices, offsets, batch: int, dense=None, more=(), inputs_ready=None) -> None:
        """``inputs_ready`` (also of step()): None = the inputs are complete in the main stream's order; "resident" =
        they already are (the ahead-work need not wait for what the main stream still has queued); an event."""
        assert self.in_flight == 0, "start() only with nothing in flight"
        for nb in [(indices, offsets, batch, dense)] + [tuple(x) for x in more]:
            b, d = self._hl_batch(nb)
            B.hl_pipe_submit(self.pipe, b, d, inputs_ready)
            self.in_flight += 1

    def step(self, grad_pop: torch.Tensor, grad_non: torch.Tensor, lr: float, next_batch=None, timers=None,
             inputs_ready=None) -> int:
        b, d = self._hl_batch(next_batch) if next_batch is not None else (None, None)
        s = B.hl_pipe_step(self.pipe, grad_pop, grad_non, lr, b, d, inputs_ready)
        self.in_flight += (1 if next_batch is not None else 0) - 1
        self.j_done += 1
        return s

    @property
    def idle(self) -> bool:
        return self.in_flight == 0

    def wait_outputs(self) -> None:
        """The main stream waits for the last write-back (device-side)."""
        B.hl_pipe_wait_outputs(self.pipe, self.main.cuda_stream)

    def wait_counts(self, stream: torch.cuda.Stream) -> None:
        """``stream`` waits until perm and counts of the mini-batch last stepped are final."""
        B.hl_pipe_wait_counts(self.pipe, stream.cuda_stream)

    def drain(self) -> None:
        B.hl_pipe_drain(self.pipe)

    def close(self) -> None:
        if getattr(self, "pipe", None):
            B.hl_pipe_drain(self.pipe)
            B.hl_pipe_destroy(self.pipe)
            self.pipe = None
        super().close()
