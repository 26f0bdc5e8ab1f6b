"""ctypes binding of libhotline.so: the same names and arguments as include/hotline.h, marshalling only.

Pointers are passed as integers (``tensor.data_ptr()``), as objects with a ``data_ptr()`` method, or None.
A negative status raises :class:`HotlineError`.  There is no fallback: if the library is missing, importing
this module fails and says how to build it.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional, Sequence

_LIB_PATH = os.path.join(os.path.dirname(os.path.abspath(__file__)), "libhotline.so")

HL_OK, HL_EINVAL, HL_EBOUNDS, HL_ECAPACITY, HL_ECUDA, HL_ETIMEOUT = 0, -1, -2, -3, -4, -5
HL_HOT_TOPK_ROWS, HL_HOT_BUDGET_BYTES, HL_HOT_FRACTION_ROWS, HL_HOT_MIN_SHARE = 0, 1, 2, 3

EXPORTS = (
    "hl_workspace_bytes", "hl_create", "hl_destroy", "hl_status", "hl_strerror", "hl_launch_count", "hl_timing_enable", "hl_timing_read", "hl_host_alloc",
    "hl_host_free", "hl_profile_hot",
    "hl_build_remap", "hl_fragment", "hl_embbag_fwd", "hl_embbag_bwd_sgd", "hl_gather_cold", "hl_scatter_cold",
    "hl_embbag_bwd_sgd_static", "hl_gather_cold_ahead", "hl_forward_cold", "hl_scatter_cold_at", "hl_flush_hot", "hl_index_cold", "hl_stage_cold", "hl_embbag_bwd_prepare", "hl_embbag_bwd_apply",
    "hl_embbag_bwd_prepare2", "hl_embbag_bwd_apply2",
    "hl_tracker_reset", "hl_tracker_update", "hl_tracker_export",
    "hl_pipe_create", "hl_pipe_create_ex", "hl_pipe_destroy", "hl_pipe_submit", "hl_pipe_step", "hl_pipe_wait_outputs", "hl_pipe_drain",
    "hl_pipe_trace_begin", "hl_pipe_trace_end", "hl_pipe_wait_counts", "hl_set_mover_ctas", "hl_test_bounded_waits", "hl_set_host_tables", "hl_set_kernel_width",
    "hl_wide_workspace_bytes", "hl_wide_create", "hl_wide_destroy", "hl_wide_status", "hl_wide_profile_hot",
    "hl_wide_build_remap", "hl_wide_fragment", "hl_wide_index_cold",
    "hl_index_cold_begin", "hl_index_cold_end", "hl_index_cold_verdict",
    "hl_embbag_bwd_prepare_merged", "hl_pipe_set_order",
)


class HotlineError(RuntimeError):
    def __init__(self, call: str, status: int):
        self.status = status
        super().__init__(f"{call} failed with status {status} ({strerror(status)})")


class hl_geometry(ctypes.Structure):
    _fields_ = [("num_tables", ctypes.c_int32), ("dim", ctypes.c_int32), ("bags_per_sample", ctypes.c_int32),
                ("table_rows", ctypes.POINTER(ctypes.c_int64))]


class hl_batch(ctypes.Structure):
    _fields_ = [("indices", ctypes.c_void_p), ("offsets", ctypes.c_void_p), ("batch", ctypes.c_int32),
                ("nnz", ctypes.c_int64)]


class hl_ubatch(ctypes.Structure):
    _fields_ = [("offsets", ctypes.c_void_p), ("ids", ctypes.c_void_p), ("cap_ids", ctypes.c_int64)]


class hl_pipe_set(ctypes.Structure):
    _fields_ = [("perm", ctypes.c_void_p), ("counts", ctypes.c_void_p), ("pop", hl_ubatch), ("non", hl_ubatch),
                ("cold_rows", ctypes.c_void_p), ("n_cold", ctypes.c_void_p), ("fwd_src", ctypes.c_void_p),
                ("pooled_pop", ctypes.c_void_p), ("pooled_non", ctypes.c_void_p), ("dense_out", ctypes.c_void_p),
                ("sorted_slots", ctypes.c_void_p), ("sorted_bags", ctypes.c_void_p), ("sorted_n", ctypes.c_void_p)]


class hl_pipe_options(ctypes.Structure):
    _fields_ = [("index_priority", ctypes.c_int32), ("link_priority", ctypes.c_int32),
                ("write_back", ctypes.c_int32)]


class hl_pipe_span(ctypes.Structure):
    _fields_ = [("mini_batch", ctypes.c_int32), ("what", ctypes.c_int32), ("stream", ctypes.c_int32),
                ("begin_ms", ctypes.c_float), ("end_ms", ctypes.c_float)]


def _load() -> ctypes.CDLL:
    if not os.path.exists(_LIB_PATH):
        raise ImportError(
            f"{_LIB_PATH} is missing: build it with `python paper_2204_05436_b200/csrc/build.py` "
            "(needs nvcc; there is no CPU fallback)")
    lib = ctypes.CDLL(_LIB_PATH)
    vp, i32, i64 = ctypes.c_void_p, ctypes.c_int32, ctypes.c_int64
    geo = ctypes.POINTER(hl_geometry)
    lib.hl_workspace_bytes.restype = ctypes.c_size_t
    lib.hl_workspace_bytes.argtypes = [geo, i32, i64, i64, i64]
    lib.hl_create.restype = i32
    lib.hl_create.argtypes = [ctypes.POINTER(vp), geo, i32, i64, i64, i64, vp, ctypes.c_size_t]
    lib.hl_destroy.restype = i32
    lib.hl_destroy.argtypes = [vp]
    lib.hl_status.restype = i32
    lib.hl_status.argtypes = [vp]
    lib.hl_strerror.restype = ctypes.c_char_p
    lib.hl_strerror.argtypes = [i32]
    lib.hl_launch_count.restype = ctypes.c_uint64
    lib.hl_launch_count.argtypes = []
    lib.hl_timing_enable.restype = i32
    lib.hl_timing_enable.argtypes = [vp, i32]
    lib.hl_timing_read.restype = i32
    lib.hl_timing_read.argtypes = [vp, i32, ctypes.POINTER(ctypes.c_float)]
    lib.hl_host_alloc.restype = vp
    lib.hl_host_alloc.argtypes = [ctypes.c_size_t]
    lib.hl_host_free.restype = i32
    lib.hl_host_free.argtypes = [vp]
    lib.hl_profile_hot.restype = i32
    lib.hl_profile_hot.argtypes = [vp, ctypes.POINTER(hl_batch), i32, i32, i32, i64, i64, vp, vp, vp]
    lib.hl_build_remap.restype = i32
    lib.hl_build_remap.argtypes = [vp, vp, vp, vp, vp, vp, vp]
    lib.hl_fragment.restype = i32
    lib.hl_fragment.argtypes = [vp, ctypes.POINTER(hl_batch), vp, i32, vp, vp, ctypes.POINTER(hl_ubatch),
                                ctypes.POINTER(hl_ubatch), vp, vp]
    lib.hl_embbag_fwd.restype = i32
    lib.hl_embbag_fwd.argtypes = [vp, vp, ctypes.POINTER(hl_ubatch), vp, vp, vp]
    lib.hl_embbag_bwd_sgd.restype = i32
    lib.hl_embbag_bwd_sgd.argtypes = [vp, vp, ctypes.POINTER(hl_ubatch), vp, vp, ctypes.c_float, vp]
    lib.hl_gather_cold.restype = i32
    lib.hl_gather_cold.argtypes = [vp, ctypes.POINTER(hl_ubatch), vp, vp, vp, vp, vp, vp]
    lib.hl_scatter_cold.restype = i32
    lib.hl_scatter_cold.argtypes = [vp, vp, vp, vp, vp, vp]
    lib.hl_gather_cold_ahead.restype = i32
    lib.hl_gather_cold_ahead.argtypes = [vp, ctypes.POINTER(hl_ubatch), vp, vp, vp, i64, i64, vp, vp, vp, vp, vp, vp, vp, vp,
                                         vp]
    lib.hl_forward_cold.restype = i32
    lib.hl_forward_cold.argtypes = [vp, vp, i64, i64, i64, vp, vp, vp]
    lib.hl_scatter_cold_at.restype = i32
    lib.hl_scatter_cold_at.argtypes = [vp, vp, i64, i64, vp, vp, vp, vp]
    lib.hl_index_cold.restype = i32
    lib.hl_index_cold.argtypes = [vp, ctypes.POINTER(hl_ubatch), vp, i64, i64, vp, vp, vp, vp, vp, vp]
    lib.hl_stage_cold.restype = i32
    lib.hl_stage_cold.argtypes = [vp, vp, vp, i64, i64, vp, vp, vp, vp]
    lib.hl_embbag_bwd_prepare.restype = i32
    lib.hl_embbag_bwd_prepare.argtypes = [vp, ctypes.POINTER(hl_ubatch), vp, vp, vp, vp, vp]
    lib.hl_embbag_bwd_apply.restype = i32
    lib.hl_embbag_bwd_apply.argtypes = [vp, vp, vp, vp, vp, vp, ctypes.c_float, vp]
    lib.hl_embbag_bwd_prepare2.restype = i32
    lib.hl_embbag_bwd_prepare2.argtypes = [vp, ctypes.POINTER(hl_ubatch), vp, ctypes.POINTER(hl_ubatch), vp, vp, vp, vp, vp]
    lib.hl_embbag_bwd_apply2.restype = i32
    lib.hl_embbag_bwd_apply2.argtypes = [vp, vp, vp, vp, vp, i32, vp, ctypes.c_float, vp]
    lib.hl_tracker_reset.restype = i32
    lib.hl_tracker_reset.argtypes = [vp, vp, vp, i64, i32, vp, vp]
    lib.hl_tracker_update.restype = i32
    lib.hl_tracker_update.argtypes = [vp, ctypes.POINTER(hl_batch), vp, vp, i64, i32, vp, vp]
    lib.hl_tracker_export.restype = i32
    lib.hl_tracker_export.argtypes = [vp, vp, vp, i64, i32, vp]
    lib.hl_pipe_create.restype = vp
    lib.hl_pipe_create.argtypes = [vp, vp, vp, i64, i32, ctypes.POINTER(hl_pipe_set), i32, vp]
    lib.hl_pipe_destroy.restype = None
    lib.hl_pipe_destroy.argtypes = [vp]
    lib.hl_pipe_submit.restype = i32
    lib.hl_pipe_submit.argtypes = [vp, ctypes.POINTER(hl_batch), vp, vp]
    lib.hl_pipe_step.restype = i32
    lib.hl_pipe_step.argtypes = [vp, vp, vp, ctypes.c_float, ctypes.POINTER(hl_batch), vp, vp, ctypes.POINTER(i32)]
    lib.hl_pipe_wait_outputs.restype = i32
    lib.hl_pipe_wait_outputs.argtypes = [vp, vp]
    lib.hl_pipe_drain.restype = i32
    lib.hl_pipe_drain.argtypes = [vp]
    lib.hl_index_cold_begin.restype = i32
    lib.hl_index_cold_begin.argtypes = [vp, ctypes.POINTER(hl_ubatch), vp, i64, i64, vp, vp, vp]
    lib.hl_index_cold_verdict.restype = vp
    lib.hl_index_cold_verdict.argtypes = [vp]
    lib.hl_index_cold_end.restype = i32
    lib.hl_index_cold_end.argtypes = [vp, ctypes.POINTER(hl_ubatch), i64, i64, vp, vp, vp, vp, vp, i32, vp]
    lib.hl_embbag_bwd_prepare_merged.restype = i32
    lib.hl_embbag_bwd_prepare_merged.argtypes = [vp, ctypes.POINTER(hl_ubatch), vp, ctypes.POINTER(hl_ubatch), vp, vp, vp, vp, vp]
    lib.hl_pipe_set_order.restype = i32
    lib.hl_pipe_set_order.argtypes = [vp, i32]
    lib.hl_pipe_wait_counts.restype = i32
    lib.hl_pipe_wait_counts.argtypes = [vp, vp]
    lib.hl_pipe_create_ex.restype = vp
    lib.hl_pipe_create_ex.argtypes = [vp, vp, vp, i64, i32, ctypes.POINTER(hl_pipe_set), i32, vp,
                                      ctypes.POINTER(hl_pipe_options)]
    lib.hl_pipe_trace_begin.restype = i32
    lib.hl_pipe_trace_begin.argtypes = [vp, i32, ctypes.c_uint32]
    lib.hl_pipe_trace_end.restype = i32
    lib.hl_pipe_trace_end.argtypes = [vp, ctypes.POINTER(hl_pipe_span), i32, ctypes.POINTER(i32)]
    lib.hl_set_mover_ctas.restype = i32
    lib.hl_set_mover_ctas.argtypes = [vp, i32, i32]
    lib.hl_wide_workspace_bytes.restype = ctypes.c_size_t
    lib.hl_wide_workspace_bytes.argtypes = [geo, i32, i64, i64, i64, i64]
    lib.hl_wide_create.restype = i32
    lib.hl_wide_create.argtypes = [ctypes.POINTER(vp), geo, i32, i64, i64, i64, i64, vp, ctypes.c_size_t]
    lib.hl_wide_destroy.restype = i32
    lib.hl_wide_destroy.argtypes = [vp]
    lib.hl_wide_status.restype = i32
    lib.hl_wide_status.argtypes = [vp]
    lib.hl_wide_profile_hot.restype = i32
    lib.hl_wide_profile_hot.argtypes = [vp, ctypes.POINTER(hl_batch), i32, i32, i32, i64, i64, i32, vp, vp, vp]
    lib.hl_wide_build_remap.restype = i32
    lib.hl_wide_build_remap.argtypes = [vp, vp, vp, vp]
    lib.hl_wide_fragment.restype = i32
    lib.hl_wide_fragment.argtypes = [vp, ctypes.POINTER(hl_batch), vp, vp, ctypes.POINTER(hl_ubatch), vp, vp, i64, vp]
    lib.hl_wide_index_cold.restype = i32
    lib.hl_wide_index_cold.argtypes = [vp, vp, vp, i64, vp, vp, vp, vp, vp]
    lib.hl_set_kernel_width.restype = i32
    lib.hl_set_kernel_width.argtypes = [vp, i32, i32]
    lib.hl_set_host_tables.restype = i32
    lib.hl_set_host_tables.argtypes = [vp, ctypes.POINTER(vp)]
    lib.hl_test_bounded_waits.restype = i32
    lib.hl_test_bounded_waits.argtypes = [vp, i32, i64]
    lib.hl_flush_hot.restype = i32
    lib.hl_flush_hot.argtypes = [vp, vp, vp, vp, vp, vp]
    lib.hl_embbag_bwd_sgd_static.restype = i32
    lib.hl_embbag_bwd_sgd_static.argtypes = [vp, i64, i32, vp, vp, i32, i64, vp, ctypes.c_float, vp, vp]
    return lib


_lib = _load()


def library_path() -> str:
    return _LIB_PATH


def _ptr(x) -> Optional[int]:
    if x is None:
        return None
    if isinstance(x, int):
        return x
    return int(x.data_ptr())


def _check(call: str, status: int) -> int:
    if status < 0:
        raise HotlineError(call, status)
    return status


def strerror(status: int) -> str:
    return _lib.hl_strerror(int(status)).decode()


def hl_launch_count() -> int:
    return int(_lib.hl_launch_count())


HL_TIMER_GATHER_MOVE, HL_TIMER_SCATTER_MOVE, HL_TIMER_BWD_REDUCE, HL_TIMER_FWD = 0, 1, 2, 3


def hl_timing_enable(ctx: int, on: bool) -> None:
    _check("hl_timing_enable", _lib.hl_timing_enable(ctx, int(on)))


def hl_timing_read(ctx: int, which: int) -> float:
    """Milliseconds of the last recorded event pair of timer ``which`` (synchronise first)."""
    ms = ctypes.c_float()
    _check("hl_timing_read", _lib.hl_timing_read(ctx, which, ctypes.byref(ms)))
    return float(ms.value)


def hl_host_alloc(nbytes: int) -> int:
    p = _lib.hl_host_alloc(int(nbytes))
    if not p:
        raise HotlineError("hl_host_alloc", HL_ECUDA)
    return int(p)


def hl_host_free(ptr: int) -> None:
    _check("hl_host_free", _lib.hl_host_free(ptr))


def host_table_tensor(n_rows: int, dim: int):
    """fp32 [n_rows, dim] torch tensor over memory from hl_host_alloc (exact size).  Free it with
    ``hl_host_free(t.data_ptr())`` once no tensor or kernel uses it any more."""
    import numpy as np
    import torch
    nbytes = int(n_rows) * int(dim) * 4
    ptr = hl_host_alloc(nbytes)
    buf = (ctypes.c_float * (int(n_rows) * int(dim))).from_address(ptr)
    return torch.from_numpy(np.frombuffer(buf, dtype=np.float32).reshape(int(n_rows), int(dim)))


def make_geometry(table_rows: Sequence[int], dim: int, bags_per_sample: int = 1) -> hl_geometry:
    arr = (ctypes.c_int64 * len(table_rows))(*[int(r) for r in table_rows])
    g = hl_geometry(len(table_rows), int(dim), int(bags_per_sample), arr)
    g._keepalive = arr
    return g


def make_batch(indices, offsets, batch: int, nnz: int) -> hl_batch:
    return hl_batch(_ptr(indices), _ptr(offsets), int(batch), int(nnz))


def make_ubatch(offsets, ids, cap_ids: int) -> hl_ubatch:
    return hl_ubatch(_ptr(offsets), _ptr(ids), int(cap_ids))


def hl_workspace_bytes(geom: hl_geometry, max_batch: int, max_nnz: int, hot_cap_rows: int,
                       staging_cap_rows: int) -> int:
    n = _lib.hl_workspace_bytes(ctypes.byref(geom), max_batch, max_nnz, hot_cap_rows, staging_cap_rows)
    if n == 0:
        raise HotlineError("hl_workspace_bytes", HL_EINVAL)
    return int(n)


def hl_create(geom: hl_geometry, max_batch: int, max_nnz: int, hot_cap_rows: int, staging_cap_rows: int,
              d_workspace, ws_bytes: int) -> int:
    ctx = ctypes.c_void_p()
    _check("hl_create", _lib.hl_create(ctypes.byref(ctx), ctypes.byref(geom), max_batch, max_nnz, hot_cap_rows,
                                       staging_cap_rows, _ptr(d_workspace), ws_bytes))
    return ctx.value


def hl_destroy(ctx: int) -> None:
    _check("hl_destroy", _lib.hl_destroy(ctx))


def hl_status(ctx: int, raise_on_error: bool = True) -> int:
    st = _lib.hl_status(ctx)
    if raise_on_error:
        _check("hl_status", st)
    return st


def hl_profile_hot(ctx: int, batch: Optional[hl_batch], reset: bool, finalize: bool, policy: int, p_num: int,
                   p_den: int, d_hot_rows, d_n_hot, stream: int) -> None:
    b = ctypes.byref(batch) if batch is not None else None
    _check("hl_profile_hot", _lib.hl_profile_hot(ctx, b, int(reset), int(finalize), policy, p_num, p_den,
                                                 _ptr(d_hot_rows), _ptr(d_n_hot), stream))


def hl_build_remap(ctx: int, d_hot_rows, d_n_hot, host_table, d_cache, d_remap_out, stream: int) -> None:
    _check("hl_build_remap", _lib.hl_build_remap(ctx, _ptr(d_hot_rows), _ptr(d_n_hot), _ptr(host_table),
                                                 _ptr(d_cache), _ptr(d_remap_out), stream))


def hl_fragment(ctx: int, batch: hl_batch, d_dense, n_dense: int, d_perm, d_counts, pop: hl_ubatch,
                non: hl_ubatch, d_dense_out, stream: int) -> None:
    _check("hl_fragment", _lib.hl_fragment(ctx, ctypes.byref(batch), _ptr(d_dense), n_dense, _ptr(d_perm),
                                           _ptr(d_counts), ctypes.byref(pop), ctypes.byref(non),
                                           _ptr(d_dense_out), stream))


def hl_embbag_fwd(ctx: int, d_cache, ub: hl_ubatch, d_n_samples, d_out, stream: int) -> None:
    _check("hl_embbag_fwd", _lib.hl_embbag_fwd(ctx, _ptr(d_cache), ctypes.byref(ub), _ptr(d_n_samples),
                                               _ptr(d_out), stream))


def hl_embbag_bwd_sgd(ctx: int, d_cache, ub: hl_ubatch, d_n_samples, d_grad_out, lr: float, stream: int) -> None:
    _check("hl_embbag_bwd_sgd", _lib.hl_embbag_bwd_sgd(ctx, _ptr(d_cache), ctypes.byref(ub), _ptr(d_n_samples),
                                                       _ptr(d_grad_out), float(lr), stream))


def hl_gather_cold(ctx: int, non: hl_ubatch, d_n_non, host_table, d_cache, d_cold_rows, d_n_cold,
                   stream: int) -> None:
    _check("hl_gather_cold", _lib.hl_gather_cold(ctx, ctypes.byref(non), _ptr(d_n_non), _ptr(host_table),
                                                 _ptr(d_cache), _ptr(d_cold_rows), _ptr(d_n_cold), stream))


def hl_scatter_cold(ctx: int, d_cache, d_cold_rows, d_n_cold, host_table, stream: int) -> None:
    _check("hl_scatter_cold", _lib.hl_scatter_cold(ctx, _ptr(d_cache), _ptr(d_cold_rows), _ptr(d_n_cold),
                                                   _ptr(host_table), stream))


HL_STATIC_MAX_NNZ, HL_STATIC_MAX_DIM = 65536, 128


def hl_embbag_bwd_sgd_static(d_cache, cache_rows: int, dim: int, d_offsets, d_ids, n_bags: int, nnz: int,
                             d_grad_out, lr: float, d_status, stream: int) -> None:
    """Backward + SGD for callers that cannot allocate device memory: no context, no workspace; the scratch is a
    fixed array inside the library (see include/hotline.h for the limits and the sharing rule)."""
    _check("hl_embbag_bwd_sgd_static", _lib.hl_embbag_bwd_sgd_static(
        _ptr(d_cache), int(cache_rows), int(dim), _ptr(d_offsets), _ptr(d_ids), int(n_bags), int(nnz),
        _ptr(d_grad_out), float(lr), _ptr(d_status), stream))


def _ev(e):
    """A torch.cuda.Event (already recorded or created with its handle), a raw cudaEvent_t as int, or None."""
    if e is None:
        return None
    if isinstance(e, int):
        return e
    return int(e.cuda_event)


def hl_gather_cold_ahead(ctx: int, non: hl_ubatch, d_n_non, host_table, d_cache, stage_row0: int, stage_rows: int,
                         d_cold_rows, d_n_cold, d_prev_cold_rows, d_n_prev, d_fwd_src, record_after_index,
                         wait_before_move_a, wait_before_move_b, stream: int) -> None:
    _check("hl_gather_cold_ahead", _lib.hl_gather_cold_ahead(
        ctx, ctypes.byref(non), _ptr(d_n_non), _ptr(host_table), _ptr(d_cache), int(stage_row0), int(stage_rows),
        _ptr(d_cold_rows), _ptr(d_n_cold), _ptr(d_prev_cold_rows), _ptr(d_n_prev), _ptr(d_fwd_src),
        _ev(record_after_index), _ev(wait_before_move_a), _ev(wait_before_move_b), stream))


def hl_forward_cold(ctx: int, d_cache, from_stage_row0: int, to_stage_row0: int, stage_rows: int, d_fwd_src, d_n_cold,
                    stream: int) -> None:
    _check("hl_forward_cold", _lib.hl_forward_cold(ctx, _ptr(d_cache), int(from_stage_row0), int(to_stage_row0),
                                                   int(stage_rows), _ptr(d_fwd_src), _ptr(d_n_cold), stream))


def hl_scatter_cold_at(ctx: int, d_cache, stage_row0: int, stage_rows: int, d_cold_rows, d_n_cold, host_table,
                       stream: int) -> None:
    _check("hl_scatter_cold_at", _lib.hl_scatter_cold_at(ctx, _ptr(d_cache), int(stage_row0), int(stage_rows),
                                                         _ptr(d_cold_rows), _ptr(d_n_cold), _ptr(host_table), stream))


def hl_flush_hot(ctx: int, d_cache, d_hot_rows, d_n_hot, host_table, stream: int) -> None:
    _check("hl_flush_hot", _lib.hl_flush_hot(ctx, _ptr(d_cache), _ptr(d_hot_rows), _ptr(d_n_hot), _ptr(host_table),
                                             stream))


def hl_index_cold(ctx: int, non: hl_ubatch, d_n_non, stage_row0: int, stage_rows: int, d_cold_rows, d_n_cold,
                  d_prev_cold_rows, d_n_prev, d_fwd_src, stream: int) -> None:
    _check("hl_index_cold", _lib.hl_index_cold(ctx, ctypes.byref(non), _ptr(d_n_non), int(stage_row0), int(stage_rows),
                                               _ptr(d_cold_rows), _ptr(d_n_cold), _ptr(d_prev_cold_rows), _ptr(d_n_prev),
                                               _ptr(d_fwd_src), stream))


def hl_stage_cold(ctx: int, host_table, d_cache, stage_row0: int, stage_rows: int, d_cold_rows, d_n_cold, d_fwd_src,
                  stream: int) -> None:
    _check("hl_stage_cold", _lib.hl_stage_cold(ctx, _ptr(host_table), _ptr(d_cache), int(stage_row0), int(stage_rows),
                                               _ptr(d_cold_rows), _ptr(d_n_cold), _ptr(d_fwd_src), stream))


def hl_embbag_bwd_prepare(ctx: int, ub: hl_ubatch, d_n_samples, d_sorted_slots, d_sorted_bags, d_n_lookups,
                          stream: int) -> None:
    _check("hl_embbag_bwd_prepare", _lib.hl_embbag_bwd_prepare(ctx, ctypes.byref(ub), _ptr(d_n_samples),
                                                               _ptr(d_sorted_slots), _ptr(d_sorted_bags),
                                                               _ptr(d_n_lookups), stream))


def hl_embbag_bwd_apply(ctx: int, d_cache, d_sorted_slots, d_sorted_bags, d_n_lookups, d_grad_out, lr: float,
                        stream: int) -> None:
    _check("hl_embbag_bwd_apply", _lib.hl_embbag_bwd_apply(ctx, _ptr(d_cache), _ptr(d_sorted_slots),
                                                           _ptr(d_sorted_bags), _ptr(d_n_lookups), _ptr(d_grad_out),
                                                           float(lr), stream))


def hl_embbag_bwd_prepare2(ctx: int, pop: hl_ubatch, d_n_pop, non: hl_ubatch, d_n_non, d_sorted_slots, d_sorted_bags,
                           d_n_lookups, stream: int) -> None:
    _check("hl_embbag_bwd_prepare2", _lib.hl_embbag_bwd_prepare2(
        ctx, ctypes.byref(pop), _ptr(d_n_pop), ctypes.byref(non), _ptr(d_n_non), _ptr(d_sorted_slots),
        _ptr(d_sorted_bags), _ptr(d_n_lookups), stream))


def hl_embbag_bwd_apply2(ctx: int, d_cache, d_sorted_slots, d_sorted_bags, d_n_lookups, which: int, d_grad_out,
                         lr: float, stream: int) -> None:
    _check("hl_embbag_bwd_apply2", _lib.hl_embbag_bwd_apply2(
        ctx, _ptr(d_cache), _ptr(d_sorted_slots), _ptr(d_sorted_bags), _ptr(d_n_lookups), int(which),
        _ptr(d_grad_out), float(lr), stream))


def hl_tracker_reset(ctx: int, d_tags, d_rrpv, n_sets: int, ways: int, d_hits, stream: int) -> None:
    _check("hl_tracker_reset", _lib.hl_tracker_reset(ctx, _ptr(d_tags), _ptr(d_rrpv), int(n_sets), int(ways),
                                                     _ptr(d_hits), stream))


def hl_tracker_update(ctx: int, batch: hl_batch, d_tags, d_rrpv, n_sets: int, ways: int, d_hits, stream: int) -> None:
    _check("hl_tracker_update", _lib.hl_tracker_update(ctx, ctypes.byref(batch), _ptr(d_tags), _ptr(d_rrpv),
                                                       int(n_sets), int(ways), _ptr(d_hits), stream))


def hl_tracker_export(ctx: int, d_tags, d_rrpv, n_sets: int, ways: int, stream: int) -> None:
    _check("hl_tracker_export", _lib.hl_tracker_export(ctx, _ptr(d_tags), _ptr(d_rrpv), int(n_sets), int(ways),
                                                       stream))


def hl_pipe_create(ctx: int, d_cache, host_table, window_rows: int, sets, n_dense: int, main_stream: int) -> int:
    """``sets``: a list of hl_pipe_set.  Returns the pipeline handle."""
    arr = (hl_pipe_set * len(sets))(*sets)
    p = _lib.hl_pipe_create(ctx, _ptr(d_cache), _ptr(host_table), int(window_rows), len(sets), arr, int(n_dense),
                            main_stream)
    if not p:
        raise HotlineError("hl_pipe_create", HL_EINVAL)
    return p


def hl_pipe_create_ex(ctx: int, d_cache, host_table, window_rows: int, sets, n_dense: int, main_stream: int,
                      index_priority: int = 0, link_priority: int = 0, write_back: int = 0) -> int:
    """hl_pipe_create with its options: the stream priorities of the ahead-work and of the host-link transfers, and
    when a mini-batch's write-back runs (HL_PIPE_WB_*)."""
    arr = (hl_pipe_set * len(sets))(*sets)
    opt = hl_pipe_options(int(index_priority), int(link_priority), int(write_back))
    p = _lib.hl_pipe_create_ex(ctx, _ptr(d_cache), _ptr(host_table), int(window_rows), len(sets), arr, int(n_dense),
                               main_stream, ctypes.byref(opt))
    if not p:
        raise HotlineError("hl_pipe_create_ex", HL_EINVAL)
    return p


def hl_set_mover_ctas(ctx: int, read_ctas: int, write_ctas: int) -> None:
    _check("hl_set_mover_ctas", _lib.hl_set_mover_ctas(ctx, int(read_ctas), int(write_ctas)))


def hl_wide_workspace_bytes(geom: hl_geometry, max_batch: int, max_nnz: int, hot_cap_rows: int, staging_cap_rows: int,
                            counter_slots: int) -> int:
    n = _lib.hl_wide_workspace_bytes(ctypes.byref(geom), max_batch, max_nnz, hot_cap_rows, staging_cap_rows,
                                     counter_slots)
    if n == 0:
        raise HotlineError("hl_wide_workspace_bytes", HL_EINVAL)
    return int(n)


def hl_wide_create(geom: hl_geometry, max_batch: int, max_nnz: int, hot_cap_rows: int, staging_cap_rows: int,
                   counter_slots: int, d_workspace, ws_bytes: int) -> int:
    w = ctypes.c_void_p()
    _check("hl_wide_create", _lib.hl_wide_create(ctypes.byref(w), ctypes.byref(geom), max_batch, max_nnz, hot_cap_rows,
                                                 staging_cap_rows, counter_slots, _ptr(d_workspace), ws_bytes))
    return w.value


def hl_wide_destroy(w: int) -> None:
    _check("hl_wide_destroy", _lib.hl_wide_destroy(w))


def hl_wide_status(w: int, raise_on_error: bool = True) -> int:
    st = _lib.hl_wide_status(w)
    if raise_on_error:
        _check("hl_wide_status", st)
    return st


def hl_wide_profile_hot(w: int, batch: Optional[hl_batch], reset: bool, finalize: bool, policy: int, p_num: int,
                        p_den: int, row_bytes: int, d_hot_rows, d_n_hot, stream: int) -> None:
    b = ctypes.byref(batch) if batch is not None else None
    _check("hl_wide_profile_hot", _lib.hl_wide_profile_hot(w, b, int(reset), int(finalize), policy, p_num, p_den,
                                                           int(row_bytes), _ptr(d_hot_rows), _ptr(d_n_hot), stream))


def hl_wide_build_remap(w: int, d_hot_rows, d_n_hot, stream: int) -> None:
    _check("hl_wide_build_remap", _lib.hl_wide_build_remap(w, _ptr(d_hot_rows), _ptr(d_n_hot), stream))


def hl_wide_fragment(w: int, batch: hl_batch, d_perm, d_counts, pop: hl_ubatch, d_non_offsets, d_non_rows,
                     non_cap: int, stream: int) -> None:
    _check("hl_wide_fragment", _lib.hl_wide_fragment(w, ctypes.byref(batch), _ptr(d_perm), _ptr(d_counts),
                                                     ctypes.byref(pop), _ptr(d_non_offsets), _ptr(d_non_rows),
                                                     int(non_cap), stream))


def hl_wide_index_cold(w: int, d_non_offsets, d_non_rows, non_cap: int, d_n_non, d_non_slots, d_cold_rows, d_n_cold,
                       stream: int) -> None:
    _check("hl_wide_index_cold", _lib.hl_wide_index_cold(w, _ptr(d_non_offsets), _ptr(d_non_rows), int(non_cap),
                                                         _ptr(d_n_non), _ptr(d_non_slots), _ptr(d_cold_rows),
                                                         _ptr(d_n_cold), stream))


def hl_set_kernel_width(ctx: int, fwd_ctas_per_sm: int, bwd_ctas_per_sm: int) -> None:
    _check("hl_set_kernel_width", _lib.hl_set_kernel_width(ctx, int(fwd_ctas_per_sm), int(bwd_ctas_per_sm)))


def hl_set_host_tables(ctx: int, tables) -> None:
    """``tables``: one device-addressable fp32 [rows_t, D] tensor (or address) per table, or None for a single table."""
    if tables is None:
        _check("hl_set_host_tables", _lib.hl_set_host_tables(ctx, None))
        return
    arr = (ctypes.c_void_p * len(tables))(*[_ptr(t) for t in tables])
    _check("hl_set_host_tables", _lib.hl_set_host_tables(ctx, arr))


def hl_test_bounded_waits(ctx: int, poll_limit: int, stall_tile: int = -1) -> None:
    _check("hl_test_bounded_waits", _lib.hl_test_bounded_waits(ctx, int(poll_limit), int(stall_tile)))


def hl_pipe_destroy(pipe: int) -> None:
    _lib.hl_pipe_destroy(pipe)


HL_PIPE_INPUTS_RESIDENT = ctypes.c_void_p(-1).value


def _ready(inputs_ready):
    """None (main-stream order), "resident", a torch.cuda.Event or a raw cudaEvent_t."""
    if inputs_ready is None:
        return None
    if isinstance(inputs_ready, str):
        assert inputs_ready == "resident"
        return HL_PIPE_INPUTS_RESIDENT
    return _ev(inputs_ready)


def hl_pipe_submit(pipe: int, batch: hl_batch, d_dense, inputs_ready=None) -> None:
    _check("hl_pipe_submit", _lib.hl_pipe_submit(pipe, ctypes.byref(batch), _ptr(d_dense), _ready(inputs_ready)))


def hl_pipe_step(pipe: int, d_grad_pop, d_grad_non, lr: float, next_batch: Optional[hl_batch], d_next_dense,
                 next_inputs_ready=None) -> int:
    """Returns the index of the buffer set that holds the stepped mini-batch's outputs."""
    out = ctypes.c_int32(-1)
    _check("hl_pipe_step", _lib.hl_pipe_step(pipe, _ptr(d_grad_pop), _ptr(d_grad_non), float(lr),
                                             ctypes.byref(next_batch) if next_batch is not None else None,
                                             _ptr(d_next_dense), _ready(next_inputs_ready), ctypes.byref(out)))
    return int(out.value)


def hl_pipe_wait_outputs(pipe: int, stream: int) -> None:
    _check("hl_pipe_wait_outputs", _lib.hl_pipe_wait_outputs(pipe, stream))


def hl_pipe_drain(pipe: int) -> None:
    _check("hl_pipe_drain", _lib.hl_pipe_drain(pipe))


HL_SPAN_NAMES = {0: "fragment", 1: "index_begin", 2: "index_end", 3: "sort", 4: "stage_cold", 5: "forward_cold",
                 6: "fwd_pop", 7: "bwd_pop", 8: "fwd_non", 9: "bwd_non", 10: "scatter_cold",
                 16: "k_move_read", 17: "k_move_write", 18: "k_bwd_chunks", 19: "k_embbag_fwd"}
HL_SPAN_KERNEL = 16
HL_SPAN_ALL = 0xFFFFFFFF


def hl_pipe_trace_begin(pipe: int, max_spans: int, what_mask: int = HL_SPAN_ALL) -> None:
    _check("hl_pipe_trace_begin", _lib.hl_pipe_trace_begin(pipe, int(max_spans), int(what_mask) & 0xFFFFFFFF))


def hl_pipe_trace_end(pipe: int, cap: int):
    """Waits for everything queued; returns the recorded spans as dicts (times in milliseconds from the first one)."""
    arr = (hl_pipe_span * max(1, int(cap)))()
    n = ctypes.c_int32(0)
    _check("hl_pipe_trace_end", _lib.hl_pipe_trace_end(pipe, arr, int(cap), ctypes.byref(n)))
    return [dict(mini_batch=int(a.mini_batch), what=int(a.what), name=HL_SPAN_NAMES.get(int(a.what), str(a.what)),
                 stream=int(a.stream), begin_ms=float(a.begin_ms), end_ms=float(a.end_ms)) for a in arr[: n.value]]


def hl_pipe_wait_counts(pipe: int, stream: int) -> None:
    _check("hl_pipe_wait_counts", _lib.hl_pipe_wait_counts(pipe, stream))


def hl_index_cold_begin(ctx: int, non: hl_ubatch, d_n_non, stage_row0: int, stage_rows: int, d_cold_rows, d_n_cold,
                        stream: int) -> None:
    _check("hl_index_cold_begin", _lib.hl_index_cold_begin(ctx, ctypes.byref(non), _ptr(d_n_non), int(stage_row0),
                                                           int(stage_rows), _ptr(d_cold_rows), _ptr(d_n_cold), stream))


def hl_index_cold_verdict(ctx: int) -> int:
    """Device address of the verdict word (int32) of the last hl_index_cold_begin."""
    return int(_lib.hl_index_cold_verdict(ctx) or 0)


def hl_index_cold_end(ctx: int, non: hl_ubatch, stage_row0: int, stage_rows: int, d_cold_rows, d_n_cold, d_prev_cold_rows,
                      d_n_prev, d_fwd_src, general_not_needed: bool, stream: int) -> None:
    _check("hl_index_cold_end", _lib.hl_index_cold_end(ctx, ctypes.byref(non), int(stage_row0), int(stage_rows),
                                                       _ptr(d_cold_rows), _ptr(d_n_cold), _ptr(d_prev_cold_rows),
                                                       _ptr(d_n_prev), _ptr(d_fwd_src), int(bool(general_not_needed)),
                                                       stream))


HL_PIPE_ORDER_FIG8, HL_PIPE_ORDER_EQ5 = 0, 1
HL_PIPE_WB_OVERLAP, HL_PIPE_WB_EXCLUSIVE, HL_PIPE_WB_AFTER_FORWARD = 0, 1, 2


def hl_embbag_bwd_prepare_merged(ctx: int, pop: hl_ubatch, d_n_pop, non: hl_ubatch, d_n_non, d_sorted_slots,
                                 d_sorted_bags, d_n_lookups, stream: int) -> None:
    _check("hl_embbag_bwd_prepare_merged", _lib.hl_embbag_bwd_prepare_merged(
        ctx, ctypes.byref(pop), _ptr(d_n_pop), ctypes.byref(non), _ptr(d_n_non), _ptr(d_sorted_slots),
        _ptr(d_sorted_bags), _ptr(d_n_lookups), stream))


def hl_pipe_set_order(pipe: int, order: int) -> None:
    _check("hl_pipe_set_order", _lib.hl_pipe_set_order(pipe, int(order)))
