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
                 device: str = "cuda:0"):
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
        if host_table.dtype != torch.float32 or tuple(host_table.shape) != (self.N, self.D):
            raise ValueError("host_table must be fp32 [N, D]")
        if not (host_table.is_cuda or host_table.is_pinned()):
            raise ValueError("host_table must be pinned host memory (or device memory)")
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
        self.main = torch.cuda.Stream(device=dev)
        self.side = torch.cuda.Stream(device=dev)
        self.ev_frag = torch.cuda.Event()
        self.ev_gather = torch.cuda.Event()
        self.ev_pop_done = torch.cuda.Event()
        self.ctx = B.hl_create(self.geom, self.max_batch, self.max_nnz, self.hot_cap, self.staging_cap,
                               self.workspace, self.ws_bytes)

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

    # ---- acceleration phase: single calls ---------------------------------------------------------------------
    def fragment(self, indices, offsets, batch: int, dense: Optional[torch.Tensor] = None) -> None:
        B.hl_fragment(self.ctx, self._batch(indices, offsets, batch), dense, self.n_dense if dense is not None else 0,
                      self.perm, self.counts, self.pop, self.non, self.dense_out if dense is not None else None,
                      self.main.cuda_stream)

    def gather_cold(self, stream: Optional[torch.cuda.Stream] = None) -> None:
        s = stream or self.main
        B.hl_gather_cold(self.ctx, self.non, self.counts[1:], self.host_table, self.cache, self.cold_rows,
                         self.n_cold, s.cuda_stream)

    def fwd_pop(self) -> None:
        B.hl_embbag_fwd(self.ctx, self.cache, self.pop, self.counts, self.pooled_pop, self.main.cuda_stream)

    def fwd_non(self) -> None:
        B.hl_embbag_fwd(self.ctx, self.cache, self.non, self.counts[1:], self.pooled_non, self.main.cuda_stream)

    def bwd_pop(self, grad: torch.Tensor, lr: float) -> None:
        B.hl_embbag_bwd_sgd(self.ctx, self.cache, self.pop, self.counts, grad, lr, self.main.cuda_stream)

    def bwd_non(self, grad: torch.Tensor, lr: float) -> None:
        B.hl_embbag_bwd_sgd(self.ctx, self.cache, self.non, self.counts[1:], grad, lr, self.main.cuda_stream)

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
            if timers is None:
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
