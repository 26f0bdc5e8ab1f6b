"""CPU oracle for the Hotline hot path -- TEST INFRASTRUCTURE, not part of the product.

Only the tests, the smoke check and the benchmark's CPU-baseline leg may import this file.  It shares no code
with the CUDA library and never imports it.  Every function is the plain definition of one step of the
path, written with numpy in the order the paper describes the step, single-threaded, with no blocking,
fusion or reordering.  Floating-point sums are accumulated in fp64 and rounded once to fp32 (the paper
trains in full precision, i.e. fp32 storage; fp64 accumulation makes the oracle the exact result rounded).

Notation follows the paper: a mini-batch M of n inputs is split into the popular micro-batch O (l inputs)
and the non-popular micro-batch X (k inputs), Section IV-A, Eq. 3.  T tables, R_t rows in table t,
base_t = sum_{u<t} R_u, N = sum R_t, D columns, B inputs per mini-batch, S bags per input and table
(21 time steps for the time-series model, else 1).  A mini-batch is table-major CSR: bag
beta(t, b, s) = (t*B + b)*S + s holds the table-local indices indices[offsets[beta] : offsets[beta+1]].
Global row id of a lookup: g = base_t + index.

Parity pins (tests/test_oracle_*.py): brute-force loops on tiny inputs, exhaustive hot sets, the partition
identity of Eq. 3, closed-form all-hit probability under the Zipf law, integer-valued exactness,
conservation of the update, library cross-checks (torch embedding_bag, np.add.at, np.bincount).
Nothing in this file is "parity unpinned".
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import Iterable, Optional, Sequence

import numpy as np


# ----------------------------------------------------------------------------------------------------------
# helpers: bag bookkeeping of a table-major CSR mini-batch
# ----------------------------------------------------------------------------------------------------------
def table_base(table_rows: Sequence[int]) -> np.ndarray:
    """base[t] = first global row of table t, base[T] = N (Data Dispatcher address registers, Section V-A)."""
    return np.concatenate([[0], np.cumsum(np.asarray(table_rows, dtype=np.int64))]).astype(np.int64)


def lookups_of(indices, offsets, batch: int, table_rows, bags_per_sample: int = 1):
    """Per lookup j: global row g_j, bag beta_j, input (sample) b_j, table t_j."""
    indices = np.asarray(indices, dtype=np.int64)
    offsets = np.asarray(offsets, dtype=np.int64)
    T, B, S = len(table_rows), int(batch), int(bags_per_sample)
    n_bags = T * B * S
    assert offsets.shape[0] == n_bags + 1 and offsets[0] == 0 and offsets[-1] == indices.shape[0]
    sizes = np.diff(offsets)
    assert (sizes >= 0).all()
    bag = np.repeat(np.arange(n_bags, dtype=np.int64), sizes)
    t = bag // (B * S)
    b = (bag // S) % B
    g = table_base(table_rows)[t] + indices
    return g, bag, b, t


# ----------------------------------------------------------------------------------------------------------
# learning phase: access counts and the popular-row set
# ----------------------------------------------------------------------------------------------------------
def access_counts(batches: Iterable, batch: int, table_rows, bags_per_sample: int = 1) -> np.ndarray:
    """cnt[g] = number of lookups of global row g over the profiled mini-batches; every occurrence counts,
    also repeats inside one bag (the access logger keeps a per-row access frequency, Section V-B; this is
    the exact counter the paper calls the Oracle LFU logger)."""
    N = int(np.sum(np.asarray(table_rows, dtype=np.int64)))
    rows = [np.zeros(0, dtype=np.int64)]
    for indices, offsets in batches:
        g, _, _, _ = lookups_of(indices, offsets, batch, table_rows, bags_per_sample)
        assert ((np.asarray(indices) >= 0)).all() and (g < N).all()
        rows.append(g)
    return np.bincount(np.concatenate(rows), minlength=N).astype(np.int64)


def select_hot(cnt: np.ndarray, k_max: int, min_share: Optional[tuple] = None) -> np.ndarray:
    """Popular rows, ascending by global id.

    Candidates are rows seen at least once (a never-seen row is never popular).  They are ranked by
    (count descending, global id ascending) -- one ranking across all tables, as the logger is one shared
    structure -- and the first ``k_max`` are kept.  ``min_share = (num, den)`` additionally requires
    cnt[g] / total >= num / den, evaluated in exact integer arithmetic (the paper's criterion is a row that
    receives at least 1 in every 100,000 accesses, Fig. 4 caption).
    """
    cnt = np.asarray(cnt, dtype=np.int64)
    cand = np.flatnonzero(cnt >= 1)
    if min_share is not None:
        num, den = int(min_share[0]), int(min_share[1])
        total = int(cnt.sum())
        # cnt*den >= total*num  <=>  cnt >= ceil(total*num/den); Python integers, so no overflow
        c_min = -((-total * num) // den)
        cand = cand[cnt[cand] >= c_min]
    order = np.lexsort((cand, -cnt[cand]))          # primary: count descending; secondary: id ascending
    chosen = cand[order[: max(0, int(k_max))]]
    return np.sort(chosen).astype(np.int64)


def hot_capacity(policy: tuple, total_rows: int, dim: int) -> int:
    """Number of hot rows K a policy allows: ("topk", K); ("budget", bytes) -> floor(bytes / (4*D)), the
    budget counting fp32 row payload only; ("fraction", num, den) -> floor(N*num/den)."""
    if policy[0] == "topk":
        return int(policy[1])
    if policy[0] == "budget":
        return int(policy[1]) // (4 * dim)
    if policy[0] == "fraction":
        return (int(total_rows) * int(policy[1])) // int(policy[2])
    raise ValueError(policy)


def build_remap(hot_rows: np.ndarray, total_rows: int) -> np.ndarray:
    """remap[g] = i if hot_rows[i] == g else -1: the slot of a popular row in the HBM cache is its rank among
    the popular rows in ascending global id (the access logger holds row indices, never row values: Section V-B)."""
    hot_rows = np.asarray(hot_rows, dtype=np.int64)
    assert (np.diff(hot_rows) > 0).all()
    remap = np.full(int(total_rows), -1, dtype=np.int32)
    remap[hot_rows] = np.arange(hot_rows.shape[0], dtype=np.int32)
    return remap


def load_hot_cache(table: np.ndarray, hot_rows: np.ndarray) -> np.ndarray:
    """cache[i, :] = table[hot_rows[i], :], a bit copy (popular rows are replicated in GPU memory)."""
    return np.asarray(table)[np.asarray(hot_rows, dtype=np.int64)].copy()


# ----------------------------------------------------------------------------------------------------------
# acceleration phase: fragment M into O and X (Input Classifier / Lookup Engine, Sections V-A and V-C)
# ----------------------------------------------------------------------------------------------------------
@dataclass
class MicroBatch:
    samples: np.ndarray      # int64 [n]   ids (positions in M) of the inputs, ascending
    offsets: np.ndarray      # int32 [T*n*S + 1]
    ids: np.ndarray          # [L_mu]  cache slots (O, int32) or global rows (X; int64 once the model has 2^31 rows)


def _emit_microbatch(samples, per_lookup_value, offsets, T, B, S, id_dtype=np.int32) -> MicroBatch:
    """Re-lay the bags of the chosen inputs table-major, bag (t*n + i)*S + s <- bag (t*B + samples[i])*S + s,
    each bag's lookups kept in their original order."""
    samples = np.asarray(samples, dtype=np.int64)
    n = samples.shape[0]
    offsets = np.asarray(offsets, dtype=np.int64)
    tt = np.arange(T, dtype=np.int64)[:, None, None]
    ss = np.arange(S, dtype=np.int64)[None, None, :]
    src_bags = ((tt * B + samples[None, :, None]) * S + ss).reshape(-1)
    sizes = offsets[src_bags + 1] - offsets[src_bags]
    new_off = np.zeros(src_bags.shape[0] + 1, dtype=np.int64)
    np.cumsum(sizes, out=new_off[1:])
    total = int(new_off[-1])
    within = np.arange(total, dtype=np.int64) - np.repeat(new_off[:-1], sizes)
    src_pos = np.repeat(offsets[src_bags], sizes) + within
    ids = np.asarray(per_lookup_value)[src_pos].astype(id_dtype)
    return MicroBatch(samples=samples, offsets=new_off.astype(np.int32), ids=ids)


def fragment(indices, offsets, batch: int, table_rows, remap: np.ndarray, bags_per_sample: int = 1,
             dense: Optional[np.ndarray] = None):
    """Split mini-batch M into popular O and non-popular X.

    An input is popular iff *every* one of its lookups, over all tables and steps, addresses a popular row
    (a single miss makes it non-popular, Section I; the Lookup Engine checks every index of the input against
    the logger, Section V-C); an input with no lookups is vacuously popular.  O and X partition M (Eq. 3); inside
    each, inputs keep their order in M.  Returns (perm, n_pop, O, X, dense_out): perm lists O's inputs then
    X's; O.ids are cache slots, X.ids are global row ids; dense_out[i] = dense[perm[i]].
    """
    T, B, S = len(table_rows), int(batch), int(bags_per_sample)
    g, _, b, _ = lookups_of(indices, offsets, B, table_rows, S)
    slot = remap[g]
    misses = np.bincount(b[slot < 0], minlength=B)
    popular = misses == 0
    o_samples = np.flatnonzero(popular)
    x_samples = np.flatnonzero(~popular)
    perm = np.concatenate([o_samples, x_samples]).astype(np.int32)
    O = _emit_microbatch(o_samples, slot, offsets, T, B, S)
    # global row ids need 64 bits once the tables together have 2^31 rows (the paper's largest synthetic models)
    X = _emit_microbatch(x_samples, g, offsets, T, B, S, np.int64 if remap.shape[0] >= 2 ** 31 else np.int32)
    dense_out = None if dense is None else np.asarray(dense)[perm].copy()
    return perm, int(o_samples.shape[0]), O, X, dense_out


# ----------------------------------------------------------------------------------------------------------
# working set of X: cold rows staged next to the hot cache (Data Dispatcher dma_rd / gpu_rd, Section V-A)
# ----------------------------------------------------------------------------------------------------------
def gather_cold(x_rows: np.ndarray, remap: np.ndarray, hot_cap: int):
    """C = sorted distinct non-popular rows referenced by X (each staged once); unified slot of a lookup =
    its hot slot, or hot_cap + rank of its row in C.  Returns (C, slots)."""
    x_rows = np.asarray(x_rows, dtype=np.int64)
    hot_slot = remap[x_rows]
    cold = hot_slot < 0
    C = np.unique(x_rows[cold])
    slots = np.where(cold, int(hot_cap) + np.searchsorted(C, x_rows), hot_slot).astype(np.int32)
    return C.astype(np.int64), slots


def stage_cold_rows(table: np.ndarray, C: np.ndarray) -> np.ndarray:
    """staging[i, :] = table[C[i], :] (DMA read of the working parameters, bit copy)."""
    return np.asarray(table)[np.asarray(C, dtype=np.int64)].copy()


def scatter_cold(table: np.ndarray, C: np.ndarray, staging: np.ndarray) -> None:
    """table[C[i], :] = staging[i, :] (non-popular rows are updated in CPU memory by DMA write, Section IV)."""
    table[np.asarray(C, dtype=np.int64)] = staging[: len(C)]


def flush_hot(table: np.ndarray, cache: np.ndarray, hot_rows: np.ndarray) -> None:
    """table[hot_rows[i], :] = cache[i, :]: before the popular set is re-learned (the logger periodically goes
    back to its learning phase, Section V-B), the popular rows' current values return to CPU memory, the only
    place that holds every row."""
    hot_rows = np.asarray(hot_rows, dtype=np.int64)
    table[hot_rows] = cache[: len(hot_rows)]


# ----------------------------------------------------------------------------------------------------------
# embedding bag: sum pooling forward (the Reducer, Section V-D) and scatter-add + SGD backward
# ----------------------------------------------------------------------------------------------------------
def embbag_fwd(rows: np.ndarray, ids: np.ndarray, offsets: np.ndarray) -> np.ndarray:
    """out[beta, :] = sum over the bag's lookups j of rows[ids[j], :], added in lookup order in fp64 and
    rounded to fp32 once; an empty bag gives zeros; a repeated id counts each time."""
    ids = np.asarray(ids, dtype=np.int64)
    offsets = np.asarray(offsets, dtype=np.int64)
    n_bags = offsets.shape[0] - 1
    sizes = np.diff(offsets)
    acc = np.zeros((n_bags, rows.shape[1]), dtype=np.float64)
    for p in range(int(sizes.max()) if n_bags else 0):       # p-th lookup of every bag that has one
        bags = np.flatnonzero(sizes > p)
        acc[bags] += rows[ids[offsets[bags] + p]].astype(np.float64)
    return acc.astype(np.float32)


def row_gradients(ids: np.ndarray, offsets: np.ndarray, grad_out: np.ndarray):
    """Distinct ids u (ascending) and G[u, :] = sum over lookups j with ids[j] == u of grad_out[bag(j), :]
    (fp64, lookups in their stable order, with multiplicity): the gradient of sum pooling w.r.t. row u."""
    ids = np.asarray(ids, dtype=np.int64)
    offsets = np.asarray(offsets, dtype=np.int64)
    n_bags = offsets.shape[0] - 1
    bag = np.repeat(np.arange(n_bags, dtype=np.int64), np.diff(offsets))
    if ids.shape[0] == 0:
        return np.zeros(0, dtype=np.int64), np.zeros((0, grad_out.shape[1]), dtype=np.float64)
    order = np.argsort(ids, kind="stable")
    sorted_ids = ids[order]
    starts = np.flatnonzero(np.concatenate([[True], sorted_ids[1:] != sorted_ids[:-1]]))
    G = np.add.reduceat(grad_out[bag[order]].astype(np.float64), starts, axis=0)
    return sorted_ids[starts], G


def embbag_bwd_sgd(rows: np.ndarray, ids, offsets, grad_out: np.ndarray, lr: float) -> None:
    """In place: rows[u, :] <- rows[u, :] - lr * G[u, :] for every distinct id u, one update per row
    (plain SGD, no momentum or decay); rows that no lookup references keep their bits.  ``lr`` is taken at
    fp32 precision (the library receives it as a C float); arithmetic in fp64, rounded once to fp32."""
    u, G = row_gradients(ids, offsets, grad_out)
    if u.shape[0] == 0:
        return
    lr64 = float(np.float32(lr))
    rows[u] = (rows[u].astype(np.float64) - lr64 * G).astype(np.float32)


# ----------------------------------------------------------------------------------------------------------
# whole mini-batch step, with and without fragmenting
# ----------------------------------------------------------------------------------------------------------
def baseline_step(table: np.ndarray, indices, offsets, batch: int, table_rows, bags_per_sample: int,
                  grad_out: np.ndarray, lr: float) -> np.ndarray:
    """The unfragmented step the paper compares against: embedding bag over the whole mini-batch against
    the full table, then one SGD update of every touched row.  Returns pooled [T*B*S, D]; updates table."""
    g, _, _, _ = lookups_of(indices, offsets, batch, table_rows, bags_per_sample)
    pooled = embbag_fwd(table, g, offsets)
    embbag_bwd_sgd(table, g, offsets, grad_out, lr)
    return pooled


def hotline_step(table: np.ndarray, cache: np.ndarray, hot_cap: int, remap: np.ndarray, indices, offsets,
                 batch: int, table_rows, bags_per_sample: int, grad_pop: np.ndarray, grad_non: np.ndarray,
                 lr: float, deferred: bool = False):
    """One mini-batch through the pipeline of Fig. 8 (acceleration phase).

    ``cache`` is [hot_cap + staging_cap, D]: popular rows in slots [0, hot_cap), X's cold working rows staged
    from ``table`` at hot_cap + i.  Order: O forward, O backward (popular rows updated in the cache), then X
    forward and backward over cache + staging, then the staged rows written back to ``table``.  With
    ``deferred`` both forwards run before both backwards, which is the order in which the result equals
    :func:`baseline_step` exactly (the paper argues that the two micro-batches give the baseline's gradient,
    Eq. 5).  Returns (perm, n_pop, O, X, C, pooled_pop, pooled_non).
    """
    perm, n_pop, O, X, _ = fragment(indices, offsets, batch, table_rows, remap, bags_per_sample)
    C, x_slots = gather_cold(X.ids, remap, hot_cap)
    assert hot_cap + len(C) <= cache.shape[0]
    cache[hot_cap: hot_cap + len(C)] = stage_cold_rows(table, C)
    pooled_pop = embbag_fwd(cache, O.ids, O.offsets)
    if deferred:
        pooled_non = embbag_fwd(cache, x_slots, X.offsets)
        embbag_bwd_sgd(cache, O.ids, O.offsets, grad_pop, lr)
    else:
        embbag_bwd_sgd(cache, O.ids, O.offsets, grad_pop, lr)
        pooled_non = embbag_fwd(cache, x_slots, X.offsets)
    embbag_bwd_sgd(cache, x_slots, X.offsets, grad_non, lr)
    scatter_cold(table, C, cache[hot_cap: hot_cap + len(C)])
    X = MicroBatch(samples=X.samples, offsets=X.offsets, ids=x_slots)
    return perm, n_pop, O, X, C, pooled_pop, pooled_non
