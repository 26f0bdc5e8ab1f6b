"""Runs one synthetic workload through the CUDA library and through the CPU oracle, call by call, and compares.

Integer outputs (hot set, remap, perm, counts, micro-batch CSRs, cold rows, unified slots) must match bit for
bit; fp32 outputs (pooled vectors, updated rows) within rtol 1e-5 / atol 1e-6, the tolerance the benchmark spec states.
The oracle never sees a value produced by the CUDA path: both start from the same generated inputs.
"""
from __future__ import annotations

import os

import numpy as np
import torch

import gen
from oracle import hotline_oracle as orc

RTOL, ATOL = 1e-5, 1e-6


def _t(x, device):
    return torch.from_numpy(np.ascontiguousarray(x)).to(device)


def max_nnz_of(spec: gen.WorkloadSpec, geom: gen.Geometry, batch: int) -> int:
    bags = geom.num_tables * batch * geom.bags_per_sample
    return bags if spec.pooling[0] == "one" else bags * int(spec.pooling[2])


def mu_grad(grad_full, samples, T, B, S):
    """Rows of the whole-batch gradient that belong to a micro-batch's bags, in the micro-batch's bag order."""
    samples = np.asarray(samples, dtype=np.int64)
    src = ((np.arange(T)[:, None, None] * B + samples[None, :, None]) * S + np.arange(S)[None, None, :]).reshape(-1)
    return grad_full[src], src


def policy_args(policy):
    import paper_2204_05436_b200 as hl
    if policy[0] == "topk":
        return hl.HL_HOT_TOPK_ROWS, int(policy[1]), 1
    if policy[0] == "budget":
        return hl.HL_HOT_BUDGET_BYTES, int(policy[1]), 1
    if policy[0] == "fraction":
        return hl.HL_HOT_FRACTION_ROWS, int(policy[1]), int(policy[2])
    if policy[0] == "share":
        return hl.HL_HOT_MIN_SHARE, int(policy[1]), int(policy[2])
    raise ValueError(policy)


def assert_close(got, want, what):
    np.testing.assert_allclose(got, want, rtol=RTOL, atol=ATOL, err_msg=what)


def run_config_check(spec, steps: int = 1, scale_rows: float = 1.0, integer: bool = False, hot_override=None,
                     deferred: bool = False, overlap: bool = True, profile_batches=None, verbose: bool = False,
                     device: str = "cuda:0", resync: bool = True, per_table: bool = False):
    """Profiles, builds the remap, then runs ``steps`` mini-batches: the first call by call with a comparison
    after every call, the others through Hotline.step().  ``hot_override``: None (profiled), "empty", "full",
    or ("random", fraction).  With ``resync`` every step after the first starts from the oracle's tables
    (copied to the device and the host table), so that each step is a parity check on identical inputs; without
    it the two sides drift apart by their accumulated fp32 rounding.  ``per_table``: the host table is one allocation
    per table (hl_set_host_tables) instead of one for all.  Returns a dict of workload statistics."""
    import paper_2204_05436_b200 as hl

    if isinstance(spec, str):
        spec = gen.CONFIGS[spec]
    geom = gen.make_geometry(spec, scale_rows)
    T, D, S, B = geom.num_tables, geom.dim, geom.bags_per_sample, spec.batch
    N = geom.total_rows
    n_bags = T * B * S
    P = spec.profile_batches if profile_batches is None else profile_batches
    lr = 0.125 if integer else spec.lr
    max_nnz = max_nnz_of(spec, geom, B)
    K = N if spec.hot_policy[0] == "share" else orc.hot_capacity(spec.hot_policy, N, D)
    hot_cap = max(1, min(K, N))
    staging_cap = max(1, min(N, max_nnz))

    table0 = gen.table_values(np.arange(N), D, spec.seed, integer=integer)
    if per_table:
        base = geom.base
        host_table = [torch.from_numpy(table0[base[t]:base[t + 1]].copy()).pin_memory() for t in range(T)]
    else:
        host_table = torch.from_numpy(table0.copy()).pin_memory()
    h = hl.Hotline(geom.table_rows, D, S, B, max_nnz, hot_cap, staging_cap, host_table, n_dense=spec.n_dense,
                   device=device)

    def host_rows():
        return np.concatenate([t.numpy() for t in h.host_tables]) if per_table else h.host_table.numpy()

    stats = {}
    try:
        with torch.cuda.stream(h.main):
            # ---------------- learning phase ----------------
            prof = [gen.make_batch(spec, geom, i) for i in range(P)]
            cnt = orc.access_counts([(b.indices, b.offsets) for b in prof], B, geom.table_rows, S)
            if hot_override is None:
                min_share = (spec.hot_policy[1], spec.hot_policy[2]) if spec.hot_policy[0] == "share" else None
                k_sel = hot_cap if spec.hot_policy[0] == "share" else min(K, hot_cap)
                hot_o = orc.select_hot(cnt, k_sel, min_share)
                pol, p_num, p_den = policy_args(spec.hot_policy)
                for i, b in enumerate(prof):
                    h.profile(_t(b.indices, device), _t(b.offsets, device), B, reset=(i == 0))
                h.profile(None, None, reset=(P == 0), finalize=True, policy=pol, p_num=p_num, p_den=p_den)
                h.status()
                n_hot = int(h.n_hot.item())
                assert n_hot == len(hot_o), ("n_hot", n_hot, len(hot_o))
                assert np.array_equal(h.hot_rows[:n_hot].cpu().numpy(), hot_o.astype(np.int32)), "hot_rows"
            else:
                rng = np.random.default_rng(spec.seed + 99)
                if hot_override == "empty":
                    hot_o = np.zeros(0, dtype=np.int64)
                elif hot_override == "full":
                    hot_o = np.arange(min(N, hot_cap), dtype=np.int64)
                else:
                    hot_o = np.sort(rng.choice(N, int(min(hot_cap, N * hot_override[1])), replace=False)).astype(np.int64)
                h.set_hot_rows(_t(hot_o, device))
                n_hot = len(hot_o)
            remap_o = orc.build_remap(hot_o, N)
            remap_g = torch.empty(N, dtype=torch.int32, device=device)
            h.build_remap(load_rows=True, remap_out=remap_g)
            h.status()
            assert np.array_equal(remap_g.cpu().numpy(), remap_o), "remap"
            cache_o = np.zeros((hot_cap + staging_cap, D), dtype=np.float32)
            cache_o[:n_hot] = orc.load_hot_cache(table0, hot_o)
            assert np.array_equal(h.cache[:n_hot].cpu().numpy().view(np.uint32), cache_o[:n_hot].view(np.uint32)), "cache"
            table_o = table0.copy()

            # ---------------- acceleration phase ----------------
            for step in range(steps):
                bid = P + step
                if step > 0 and resync:
                    h.cache.copy_(_t(cache_o, device))
                    if per_table:
                        for t in range(T):
                            h.host_tables[t].copy_(torch.from_numpy(table_o[geom.base[t]:geom.base[t + 1]]))
                    else:
                        h.host_table.copy_(torch.from_numpy(table_o))
                    torch.cuda.synchronize()
                batch = gen.make_batch(spec, geom, bid)
                grad_full = gen.grad_values(spec.seed, bid, 2, n_bags, D, integer=integer)
                perm_o, n_pop_o, O, X, dense_o = orc.fragment(batch.indices, batch.offsets, B, geom.table_rows, remap_o, S,
                                                              batch.dense)
                g_pop, _ = mu_grad(grad_full, perm_o[:n_pop_o], T, B, S)
                g_non, _ = mu_grad(grad_full, perm_o[n_pop_o:], T, B, S)
                out = orc.hotline_step(table_o, cache_o, hot_cap, remap_o, batch.indices, batch.offsets, B,
                                       geom.table_rows, S, g_pop, g_non, lr, deferred=deferred)
                _, _, _, X_slots, C, pooled_pop_o, pooled_non_o = out
                n_non_o = B - n_pop_o
                bags_pop, bags_non = T * n_pop_o * S, T * n_non_o * S

                d_idx, d_off = _t(batch.indices, device), _t(batch.offsets, device)
                d_dense = _t(batch.dense, device) if batch.dense is not None else None
                d_gpop = torch.zeros((n_bags, D), dtype=torch.float32, device=device)
                d_gnon = torch.zeros((n_bags, D), dtype=torch.float32, device=device)
                d_gpop[:bags_pop] = _t(g_pop, device)
                d_gnon[:bags_non] = _t(g_non, device)
                torch.cuda.synchronize()

                def check_fragment():
                    counts = h.counts.cpu().numpy()
                    assert counts.tolist() == [n_pop_o, n_non_o, len(O.ids), len(X.ids)], ("counts", counts.tolist())
                    assert np.array_equal(h.perm[:B].cpu().numpy(), perm_o), "perm"
                    assert np.array_equal(h.pop_offsets[:bags_pop + 1].cpu().numpy(), O.offsets), "pop offsets"
                    assert np.array_equal(h.pop_ids[:len(O.ids)].cpu().numpy(), O.ids), "pop slots"
                    assert np.array_equal(h.non_offsets[:bags_non + 1].cpu().numpy(), X.offsets), "non offsets"
                    if dense_o is not None:
                        assert np.array_equal(h.dense_out[:B].cpu().numpy().view(np.uint32), dense_o.view(np.uint32)), "dense"

                def check_gather():
                    assert int(h.n_cold.item()) == len(C), ("n_cold", int(h.n_cold.item()), len(C))
                    assert np.array_equal(h.cold_rows[:len(C)].cpu().numpy(), C.astype(np.int32)), "cold rows"
                    assert np.array_equal(h.non_ids[:len(X.ids)].cpu().numpy(), X_slots.ids), "non slots"

                if step == 0:
                    if True:
                        h.fragment(d_idx, d_off, B, d_dense)
                        h.status()
                        check_fragment()
                        assert np.array_equal(h.non_ids[:len(X.ids)].cpu().numpy(), X.ids), "non rows"
                        h.gather_cold()
                        h.status()
                        check_gather()
                        staged = h.cache[hot_cap:hot_cap + len(C)].cpu().numpy()
                        assert np.array_equal(staged.view(np.uint32), table0[C].view(np.uint32)) or step > 0, "staging"
                        h.fwd_pop()
                        if deferred:
                            h.fwd_non()
                            h.bwd_pop(d_gpop, lr)
                        else:
                            h.bwd_pop(d_gpop, lr)
                            h.fwd_non()
                        h.bwd_non(d_gnon, lr)
                        h.scatter_cold()
                        h.status()
                else:
                    h.step(d_idx, d_off, B, d_gpop, d_gnon, lr, dense=d_dense, deferred=deferred, overlap=overlap)
                    h.status()
                    check_fragment()
                    check_gather()

                pp = h.pooled_pop[:bags_pop].cpu().numpy()
                pn = h.pooled_non[:bags_non].cpu().numpy()
                assert_close(pp, pooled_pop_o, "pooled_pop")
                assert_close(pn, pooled_non_o, "pooled_non")
                assert_close(h.cache[:n_hot].cpu().numpy(), cache_o[:n_hot], "hot rows after update")
                assert_close(h.cache[hot_cap:hot_cap + len(C)].cpu().numpy(), cache_o[hot_cap:hot_cap + len(C)],
                             "staged rows after update")
                assert_close(host_rows(), table_o, "host table after scatter")
                if integer:
                    assert np.array_equal(pp, pooled_pop_o) and np.array_equal(pn, pooled_non_o), "integer pooled"
                    assert np.array_equal(h.cache[:n_hot].cpu().numpy(), cache_o[:n_hot]), "integer hot rows"
                    assert np.array_equal(host_rows(), table_o), "integer host table"
                if spec.pooling[0] == "one" and step == 0:   # a bag of one lookup is a row copy: bit-exact
                    assert np.array_equal(pp.view(np.uint32), pooled_pop_o.view(np.uint32)), "pooled_pop bits"
                # rows nobody touched keep their bits
                touched = np.zeros(N, dtype=bool)
                touched[C] = True
                assert np.array_equal(host_rows()[~touched].view(np.uint32), table0[~touched].view(np.uint32)) \
                    or step > 0, "untouched host rows"
                stats = dict(n_pop=n_pop_o, n_non=n_non_o, n_cold=len(C), n_hot=n_hot, L_pop=len(O.ids), L_non=len(X.ids),
                             batch=B, N=N)
                if verbose:
                    print(f"[{spec.name}] step {step}: {stats}")
    finally:
        h.close()
    return stats


def run_pipelined_check(spec, steps: int = 6, scale_rows: float = 1.0, integer: bool = True, profile_batches=None,
                        device: str = "cuda:0", overlap_link: bool = True, sort_ahead: bool = True,
                        combined_sort: bool = True, lookahead: int = 2, native: bool = False,
                        drain_between: bool = False, order: str = "fig8", per_table: bool = False,
                        write_back: str = "overlap"):
    """Software-pipelined CUDA path (PipelinedHotline) against the oracle processing the same mini-batches one
    after the other.  With integer data every sum is exact, so pooled vectors, the hot cache and the host table
    must agree bit for bit after any number of steps -- which they only do if rows shared by consecutive
    mini-batches are forwarded and write-backs are ordered correctly."""
    import paper_2204_05436_b200 as hl

    if isinstance(spec, str):
        spec = gen.CONFIGS[spec]
    geom = gen.make_geometry(spec, scale_rows)
    T, D, S, B = geom.num_tables, geom.dim, geom.bags_per_sample, spec.batch
    N = geom.total_rows
    n_bags = T * B * S
    P = spec.profile_batches if profile_batches is None else profile_batches
    lr = 0.125 if integer else spec.lr
    max_nnz = max_nnz_of(spec, geom, B)
    K = orc.hot_capacity(spec.hot_policy, N, D)
    hot_cap = max(1, min(K, N))
    window = max(1, min(N, max_nnz))

    table0 = gen.table_values(np.arange(N), D, spec.seed, integer=integer)
    prof = [gen.make_batch(spec, geom, i) for i in range(P)]
    cnt = orc.access_counts([(b.indices, b.offsets) for b in prof], B, geom.table_rows, S)
    hot_o = orc.select_hot(cnt, min(K, hot_cap))
    remap_o = orc.build_remap(hot_o, N)
    n_hot = len(hot_o)

    # ---- oracle: one mini-batch after the other ----
    table_o = table0.copy()
    cache_o = np.zeros((hot_cap + window, D), dtype=np.float32)
    cache_o[:n_hot] = orc.load_hot_cache(table0, hot_o)
    batches, grads, expect = [], [], []
    shared = 0
    prev_C = np.zeros(0, dtype=np.int64)
    for step in range(steps):
        bid = P + step
        batch = gen.make_batch(spec, geom, bid)
        grad_full = gen.grad_values(spec.seed, bid, 2, n_bags, D, integer=integer)
        perm_o, n_pop_o, _, _, _ = orc.fragment(batch.indices, batch.offsets, B, geom.table_rows, remap_o, S)
        g_pop, _ = mu_grad(grad_full, perm_o[:n_pop_o], T, B, S)
        g_non, _ = mu_grad(grad_full, perm_o[n_pop_o:], T, B, S)
        if order == "fig8":
            out = orc.hotline_step(table_o, cache_o, hot_cap, remap_o, batch.indices, batch.offsets, B,
                                   geom.table_rows, S, g_pop, g_non, lr)
            _, _, _, _, C, pooled_pop_o, pooled_non_o = out
        else:
            # Eq. 5: both forwards, then ONE update of every touched row with the whole mini-batch's gradient --
            # the oracle's steps put together: O's and X's lookups as one CSR over [O's bags; X's bags]
            _, _, O, X, _ = orc.fragment(batch.indices, batch.offsets, B, geom.table_rows, remap_o, S)
            C, x_slots = orc.gather_cold(X.ids, remap_o, hot_cap)
            cache_o[hot_cap: hot_cap + len(C)] = orc.stage_cold_rows(table_o, C)
            pooled_pop_o = orc.embbag_fwd(cache_o, O.ids, O.offsets)
            pooled_non_o = orc.embbag_fwd(cache_o, x_slots, X.offsets)
            ids_all = np.concatenate([O.ids, x_slots])
            offsets_all = np.concatenate([O.offsets, X.offsets[1:] + len(O.ids)])
            orc.embbag_bwd_sgd(cache_o, ids_all, offsets_all, np.concatenate([g_pop, g_non]), lr)
            orc.scatter_cold(table_o, C, cache_o[hot_cap: hot_cap + len(C)])
        shared += len(np.intersect1d(C, prev_C))
        prev_C = C
        batches.append(batch)
        grads.append((g_pop, g_non))
        expect.append((perm_o, n_pop_o, pooled_pop_o, pooled_non_o, len(C)))

    # ---- CUDA: pipelined ----
    if per_table:      # one host allocation per table (hl_set_host_tables)
        host_table = [torch.from_numpy(table0[geom.base[t]:geom.base[t + 1]].copy()).pin_memory() for t in range(T)]
    else:
        host_table = torch.from_numpy(table0.copy()).pin_memory()

    def host_rows():
        return np.concatenate([t.numpy() for t in p.host_tables]) if per_table else p.host_table.numpy()

    if native:
        p = hl.NativePipelinedHotline(geom.table_rows, D, S, B, max_nnz, hot_cap, window, host_table,
                                      n_dense=spec.n_dense, device=device, lookahead=lookahead, order=order,
                                      write_back=write_back)
    else:
        p = hl.PipelinedHotline(geom.table_rows, D, S, B, max_nnz, hot_cap, window, host_table, n_dense=spec.n_dense,
                                device=device, overlap_link=overlap_link, sort_ahead=sort_ahead,
                                combined_sort=combined_sort, lookahead=lookahead)
    got = []
    try:
        with torch.cuda.stream(p.main):
            p.set_hot_rows(_t(hot_o, device))
            p.build_remap(load_rows=True)
            d_batches = [(_t(b.indices, device), _t(b.offsets, device), B,
                          _t(b.dense, device) if b.dense is not None else None) for b in batches]
            d_grads = []
            for (g_pop, g_non) in grads:
                gp = torch.zeros((n_bags, D), dtype=torch.float32, device=device)
                gn = torch.zeros((n_bags, D), dtype=torch.float32, device=device)
                gp[:len(g_pop)] = _t(g_pop, device)
                gn[:len(g_non)] = _t(g_non, device)
                if order == "eq5":       # one array: the gradients of O's bags, then those of X's bags
                    gp[len(g_pop):len(g_pop) + len(g_non)] = _t(g_non, device)
                    gn = None
                d_grads.append((gp, gn))
            torch.cuda.synchronize()
            ahead = p.lookahead
            launches0 = hl.hl_launch_count()
            p.start(*d_batches[0], more=d_batches[1:ahead])
            for step in range(steps):
                nxt = d_batches[step + ahead] if step + ahead < steps else None
                if drain_between:
                    p.drain()        # the device has caught up: what the ahead-work found is known to the host
                s = p.step(d_grads[step][0], d_grads[step][1], lr, next_batch=nxt)
                st = p.sets[s]
                got.append((st.perm.clone(), st.counts.clone(), st.pooled_pop.clone(), st.pooled_non.clone(),
                            st.n_cold.clone()))
            p.drain()
            p.status()
            launches = hl.hl_launch_count() - launches0
        for step in range(steps):
            perm_o, n_pop_o, pooled_pop_o, pooled_non_o, n_cold_o = expect[step]
            perm_g, counts_g, pp, pn, n_cold_g = [x.cpu().numpy() for x in got[step]]
            assert counts_g[0] == n_pop_o and counts_g[1] == B - n_pop_o, ("counts", step)
            assert np.array_equal(perm_g[:B], perm_o), ("perm", step)
            assert int(n_cold_g[0]) == n_cold_o, ("n_cold", step)
            bags_pop, bags_non = T * n_pop_o * S, T * (B - n_pop_o) * S
            if integer:
                assert np.array_equal(pp[:bags_pop], pooled_pop_o), ("pooled_pop", step)
                assert np.array_equal(pn[:bags_non], pooled_non_o), ("pooled_non", step)
            else:
                assert_close(pp[:bags_pop], pooled_pop_o, f"pooled_pop step {step}")
                assert_close(pn[:bags_non], pooled_non_o, f"pooled_non step {step}")
        hot_g = p.cache[:n_hot].cpu().numpy()
        if integer:
            assert np.array_equal(hot_g, cache_o[:n_hot]), "hot cache"
            assert np.array_equal(host_rows(), table_o), "host table"
        else:
            assert_close(hot_g, cache_o[:n_hot], "hot cache")
            assert_close(host_rows(), table_o, "host table")
    finally:
        p.close()
    return dict(shared_cold_rows=shared, steps=steps, launches=int(launches))


class _HostTable:
    """The host-DRAM table of a full-size check: one allocation of device-addressable memory, or one per table
    (for a table above what a single allocation takes).  Rows are read by global id."""

    def __init__(self, hl, geom, per_table: bool):
        self.base, self.per_table = geom.base, per_table
        if per_table:
            self.tensors = [hl.host_table_tensor(r, geom.dim) for r in geom.table_rows]
        else:
            self.tensors = [hl.host_table_tensor(geom.total_rows, geom.dim)]

    def for_library(self):
        return self.tensors if self.per_table else self.tensors[0]

    def fill(self, seed, device, integer=False):
        for t, ten in enumerate(self.tensors):
            row0 = int(self.base[t]) if self.per_table else 0
            for r0 in range(0, ten.shape[0], 1 << 21):      # rows row0 + r0 ... of the whole table
                n = min(1 << 21, ten.shape[0] - r0)
                ten[r0:r0 + n].copy_(gen.table_values_torch(row0 + r0, n, ten.shape[1], seed, device, integer=integer))
        torch.cuda.synchronize()

    def rows(self, g):
        g = np.asarray(g, dtype=np.int64)
        if not self.per_table:
            return self.tensors[0].numpy()[g]
        t = np.searchsorted(self.base, g, side="right") - 1
        out = np.empty((len(g), self.tensors[0].shape[1]), dtype=np.float32)
        for tt in np.unique(t):
            sel = t == tt
            out[sel] = self.tensors[tt].numpy()[g[sel] - self.base[tt]]
        return out

    def free(self, hl):
        ptrs = [ten.data_ptr() for ten in self.tensors]
        self.tensors = []
        for ptr in ptrs:
            hl.hl_host_free(ptr)


def run_fullsize_check(spec, scale_rows: float = 1.0, n_samples: int = 1500, profile_batches=None,
                       device: str = "cuda:0", verbose: bool = False, per_table: bool = False):
    """A workload too large for an element-by-element float comparison, run in the launch configuration the
    benchmark times (Hotline.step, cold gather on the side stream).  Every integer result is compared in full
    (hot set, perm, counts, both CSRs, cold rows, unified slots); float results are compared on sampled outputs
    that the oracle's definitions give one by one: sampled pooled vectors, sampled updated hot rows, sampled
    written-back cold rows, and sampled rows nobody touched (which must keep their bits).  The host table lives in
    pinned memory and is filled on the device from the same counter hash the oracle evaluates row by row.
    ``per_table``: one host allocation per table (hl_set_host_tables)."""
    import paper_2204_05436_b200 as hl

    if isinstance(spec, str):
        spec = gen.CONFIGS[spec]
    geom = gen.make_geometry(spec, scale_rows)
    T, D, S, B = geom.num_tables, geom.dim, geom.bags_per_sample, spec.batch
    N = geom.total_rows
    n_bags = T * B * S
    P = spec.profile_batches if profile_batches is None else profile_batches
    lr = spec.lr
    max_nnz = max_nnz_of(spec, geom, B)
    K = orc.hot_capacity(spec.hot_policy, N, D)
    hot_cap = max(1, min(K, N))
    staging_cap = max(1, min(N, max_nnz))
    rng = np.random.default_rng(spec.seed + 4242)
    rows_of = lambda g: gen.table_values(np.asarray(g, dtype=np.int64), D, spec.seed)   # noqa: E731

    table = _HostTable(hl, geom, per_table)
    h = None
    try:
        table.fill(spec.seed, torch.device(device))
        probe = rng.integers(0, N, 64)
        assert np.array_equal(table.rows(probe).view(np.uint32), rows_of(probe).view(np.uint32)), "table fill"
        h = hl.Hotline(geom.table_rows, D, S, B, max_nnz, hot_cap, staging_cap, table.for_library(),
                       n_dense=spec.n_dense, device=device)
        with torch.cuda.stream(h.main):
            # ---- learning phase: full comparison ----
            prof = [gen.make_batch(spec, geom, i) for i in range(P)]
            cnt = orc.access_counts([(b.indices, b.offsets) for b in prof], B, geom.table_rows, S)
            hot_o = orc.select_hot(cnt, min(K, hot_cap))
            del cnt
            pol, p_num, p_den = policy_args(spec.hot_policy)
            for i, b in enumerate(prof):
                h.profile(_t(b.indices, device), _t(b.offsets, device), B, reset=(i == 0))
            h.profile(None, None, finalize=True, policy=pol, p_num=p_num, p_den=p_den)
            h.build_remap(load_rows=True)
            h.status()
            n_hot = int(h.n_hot.item())
            assert n_hot == len(hot_o), ("n_hot", n_hot, len(hot_o))
            assert np.array_equal(h.hot_rows[:n_hot].cpu().numpy(), hot_o.astype(np.int32)), "hot rows"
            remap_o = orc.build_remap(hot_o, N)
            pick = rng.integers(0, n_hot, n_samples)
            got = h.cache[torch.from_numpy(pick).to(device)].cpu().numpy()
            assert np.array_equal(got.view(np.uint32), rows_of(hot_o[pick]).view(np.uint32)), "hot cache load"

            # ---- one mini-batch through Hotline.step ----
            batch = gen.make_batch(spec, geom, P)
            grad = gen.grad_values(spec.seed, P, 2, n_bags, D)
            perm_o, n_pop_o, O, X, dense_o = orc.fragment(batch.indices, batch.offsets, B, geom.table_rows, remap_o,
                                                          S, batch.dense)
            C, x_slots = orc.gather_cold(X.ids, remap_o, hot_cap)
            n_non_o = B - n_pop_o
            bags_pop, bags_non = T * n_pop_o * S, T * n_non_o * S
            d_grad = _t(grad, device)
            d_dense = _t(batch.dense, device) if batch.dense is not None else None
            d_idx, d_off = _t(batch.indices, device), _t(batch.offsets, device)
            torch.cuda.synchronize()
            h.step(d_idx, d_off, B, d_grad, d_grad, lr, dense=d_dense)
            h.status()
            assert h.counts.cpu().tolist() == [n_pop_o, n_non_o, len(O.ids), len(X.ids)], "counts"
            assert np.array_equal(h.perm[:B].cpu().numpy(), perm_o), "perm"
            assert np.array_equal(h.pop_offsets[:bags_pop + 1].cpu().numpy(), O.offsets), "pop offsets"
            assert np.array_equal(h.pop_ids[:len(O.ids)].cpu().numpy(), O.ids), "pop slots"
            assert np.array_equal(h.non_offsets[:bags_non + 1].cpu().numpy(), X.offsets), "non offsets"
            assert int(h.n_cold.item()) == len(C), "n_cold"
            assert np.array_equal(h.cold_rows[:len(C)].cpu().numpy(), C.astype(np.int32)), "cold rows"
            assert np.array_equal(h.non_ids[:len(X.ids)].cpu().numpy(), x_slots), "unified slots"
            if dense_o is not None:
                assert np.array_equal(h.dense_out[:B].cpu().numpy().view(np.uint32), dense_o.view(np.uint32)), "dense"

            # ---- sampled float results ----
            lr64 = float(np.float32(lr))

            def slot_row_id(slots):   # global row behind a unified slot
                slots = np.asarray(slots, dtype=np.int64)
                return np.where(slots < hot_cap, hot_o[np.minimum(slots, n_hot - 1)], C[np.maximum(slots - hot_cap, 0)
                                                                                        % max(1, len(C))])

            def row_grad(ids, offsets, u):   # sum of grad rows of the bags whose lookups address slot u (fp64)
                pos = np.flatnonzero(ids == u)
                bags = np.searchsorted(offsets, pos, side="right") - 1
                return grad[bags].astype(np.float64).sum(axis=0)

            # rows after O's update (needed by X's forward): start from the initial values
            o_ids64, x_ids64 = O.ids.astype(np.int64), x_slots.astype(np.int64)
            touched_by_o = np.zeros(hot_cap + staging_cap, dtype=bool)
            touched_by_o[o_ids64] = True

            def value_after_o(slots):
                base = rows_of(slot_row_id(slots))
                out = base.copy()
                for i, u in enumerate(np.asarray(slots)):
                    if touched_by_o[u]:
                        out[i] = (base[i].astype(np.float64) - lr64 * row_grad(O.ids, O.offsets, u)).astype(np.float32)
                return out

            def pooled_expect(ids, offsets, bags, value_fn):
                out = np.zeros((len(bags), D), dtype=np.float32)
                for i, bag in enumerate(bags):
                    sl = ids[offsets[bag]:offsets[bag + 1]]
                    out[i] = value_fn(sl).astype(np.float64).sum(axis=0).astype(np.float32) if len(sl) else 0.0
                return out

            n_s = max(8, n_samples // 8)
            if bags_pop:
                bags = rng.integers(0, bags_pop, n_s)
                want = pooled_expect(O.ids, O.offsets, bags, lambda sl: rows_of(slot_row_id(sl)))
                got = h.pooled_pop[torch.from_numpy(bags).to(device)].cpu().numpy()
                assert_close(got, want, "sampled pooled_pop")
            if bags_non:
                bags = rng.integers(0, bags_non, n_s)
                want = pooled_expect(x_slots, X.offsets, bags, value_after_o)
                got = h.pooled_non[torch.from_numpy(bags).to(device)].cpu().numpy()
                assert_close(got, want, "sampled pooled_non")
            # updated rows: O's update then X's update, each rounded to fp32 as the oracle does step by step
            cand = np.unique(np.concatenate([o_ids64[rng.integers(0, max(1, len(o_ids64)), n_s)] if len(o_ids64) else
                                             np.zeros(0, np.int64),
                                             x_ids64[rng.integers(0, max(1, len(x_ids64)), n_s)] if len(x_ids64) else
                                             np.zeros(0, np.int64)]))
            touched_by_x = np.zeros(hot_cap + staging_cap, dtype=bool)
            touched_by_x[x_ids64] = True
            want = value_after_o(cand)
            for i, u in enumerate(cand):
                if touched_by_x[u]:
                    want[i] = (want[i].astype(np.float64) - lr64 * row_grad(x_slots, X.offsets, u)).astype(np.float32)
            hot_part = cand < hot_cap
            got_hot = h.cache[torch.from_numpy(cand[hot_part]).to(device)].cpu().numpy()
            assert_close(got_hot, want[hot_part], "sampled updated hot rows")
            cold_ids = C[cand[~hot_part] - hot_cap]
            assert_close(table.rows(cold_ids), want[~hot_part], "sampled written-back cold rows")
            assert not np.array_equal(want[hot_part], rows_of(slot_row_id(cand[hot_part]))), "update changed nothing"
            # rows nobody touched keep their bits
            idle = np.flatnonzero(~(touched_by_o[:n_hot] | touched_by_x[:n_hot]))
            idle = idle[rng.integers(0, len(idle), min(n_samples, len(idle)))] if len(idle) else idle
            got = h.cache[torch.from_numpy(idle).to(device)].cpu().numpy()
            assert np.array_equal(got.view(np.uint32), rows_of(hot_o[idle]).view(np.uint32)), "idle hot rows"
            far = rng.integers(0, N, n_samples)
            far = far[(remap_o[far] < 0) & ~np.isin(far, C)]
            assert np.array_equal(table.rows(far).view(np.uint32), rows_of(far).view(np.uint32)), "idle host rows"
            stats = dict(n_pop=n_pop_o, n_non=n_non_o, n_cold=len(C), n_hot=n_hot, N=N, batch=B)
            if verbose:
                print(f"[{spec.name} full size] {stats}")
            return stats
    finally:
        if h is not None:
            h.close()
        torch.cuda.synchronize()
        table.free(hl)


def run_native_fullsize_check(spec, steps: int = 4, scale_rows: float = 1.0, profile_batches=None, lookahead: int = 2,
                              order: str = "fig8", device: str = "cuda:0", verbose: bool = False):
    """The schedule the benchmark times (the library's own scheduler, hl_pipe_*, default lookahead and order) on a
    workload too large to hold twice, over several mini-batches, against orc.hotline_step applied in sequence.

    Integer-valued tables and gradients make every sum exact, so everything is compared bit for bit and in full:
    perm, counts, the number of cold rows, both pooled arrays of every mini-batch, the whole hot cache at the end,
    and every host row that any mini-batch wrote back; sampled host rows nobody touched must keep their bits.
    The oracle's table is a sparse file mapped into memory (same shape as the real table, same global row ids):
    only the rows the mini-batches stage are ever populated, with the values the procedural initialiser gives."""
    import tempfile

    import bench
    import paper_2204_05436_b200 as hl

    if isinstance(spec, str):
        spec = gen.CONFIGS[spec]
    geom = gen.make_geometry(spec, scale_rows)
    T, D, S, B = geom.num_tables, geom.dim, geom.bags_per_sample, spec.batch
    N = geom.total_rows
    n_bags = T * B * S
    P = spec.profile_batches if profile_batches is None else profile_batches
    lr = 0.125
    max_nnz = max_nnz_of(spec, geom, B)
    K = orc.hot_capacity(spec.hot_policy, N, D)
    hot_cap = max(1, min(K, N))
    window = max(1, min(N, max_nnz))
    rng = np.random.default_rng(spec.seed + 777)
    rows_of = lambda g: gen.table_values(np.asarray(g, dtype=np.int64), D, spec.seed, integer=True)   # noqa: E731

    table = hl.host_table_tensor(N, D)
    p, table_o = None, None
    tmp = tempfile.TemporaryDirectory()
    try:
        bench.fill_table(table, D, spec.seed, torch.device(device), integer=True)
        probe = rng.integers(0, N, 64)
        assert np.array_equal(table.numpy()[probe], rows_of(probe)), "table fill"

        # ---- oracle: learning phase, then the mini-batches one after the other on the sparse table ----
        prof = [gen.make_batch(spec, geom, i) for i in range(P)]
        cnt = orc.access_counts([(b.indices, b.offsets) for b in prof], B, geom.table_rows, S)
        hot_o = orc.select_hot(cnt, min(K, hot_cap))
        del cnt
        n_hot = len(hot_o)
        remap_o = orc.build_remap(hot_o, N)
        batches = [gen.make_batch(spec, geom, P + i) for i in range(steps)]
        table_o = np.memmap(os.path.join(tmp.name, "oracle_table.f32"), dtype=np.float32, mode="w+", shape=(N, D))
        staged_rows = np.zeros(0, dtype=np.int64)
        for b in batches:                       # index-only pass: which rows will ever be staged
            _, _, _, X, _ = orc.fragment(b.indices, b.offsets, B, geom.table_rows, remap_o, S)
            C, _ = orc.gather_cold(X.ids, remap_o, hot_cap)
            staged_rows = np.union1d(staged_rows, C)
        table_o[staged_rows] = rows_of(staged_rows)
        cache_o = np.zeros((hot_cap + window, D), dtype=np.float32)
        cache_o[:n_hot] = rows_of(hot_o)
        grads, expect, shared, prev_C = [], [], 0, np.zeros(0, dtype=np.int64)
        for i, b in enumerate(batches):
            grad_full = gen.grad_values(spec.seed, P + i, 2, n_bags, D, integer=True)
            perm_o, n_pop_o, _, _, _ = orc.fragment(b.indices, b.offsets, B, geom.table_rows, remap_o, S)
            g_pop, _ = mu_grad(grad_full, perm_o[:n_pop_o], T, B, S)
            g_non, _ = mu_grad(grad_full, perm_o[n_pop_o:], T, B, S)
            out = orc.hotline_step(table_o, cache_o, hot_cap, remap_o, b.indices, b.offsets, B, geom.table_rows, S,
                                   g_pop, g_non, lr, deferred=(order == "eq5"))
            _, _, O, X, C, pooled_pop_o, pooled_non_o = out
            shared += len(np.intersect1d(C, prev_C))
            prev_C = C
            grads.append((g_pop, g_non))
            expect.append((perm_o, n_pop_o, len(O.ids), len(X.ids), len(C), pooled_pop_o, pooled_non_o))

        # ---- CUDA: the library's scheduler ----
        p = hl.NativePipelinedHotline(geom.table_rows, D, S, B, max_nnz, hot_cap, window, table, n_dense=spec.n_dense,
                                      device=device, lookahead=lookahead, order=order)
        with torch.cuda.stream(p.main):
            pol, p_num, p_den = policy_args(spec.hot_policy)
            for i, b in enumerate(prof):
                p.profile(_t(b.indices, device), _t(b.offsets, device), B, reset=(i == 0))
            p.profile(None, None, finalize=True, policy=pol, p_num=p_num, p_den=p_den)
            p.build_remap(load_rows=True)
            p.status()
            assert int(p.n_hot.item()) == n_hot, ("n_hot", int(p.n_hot.item()), n_hot)
            assert np.array_equal(p.hot_rows[:n_hot].cpu().numpy(), hot_o.astype(np.int32)), "hot rows"
            del prof
            d_batches = [(_t(b.indices, device), _t(b.offsets, device), B,
                          _t(b.dense, device) if b.dense is not None else None) for b in batches]
            d_grads = []
            for (g_pop, g_non) in grads:
                gp = torch.zeros((n_bags, D), dtype=torch.float32, device=device)
                gp[:len(g_pop)] = _t(g_pop, device)
                if order == "eq5":
                    gp[len(g_pop):len(g_pop) + len(g_non)] = _t(g_non, device)
                    gn = None
                else:
                    gn = torch.zeros((n_bags, D), dtype=torch.float32, device=device)
                    gn[:len(g_non)] = _t(g_non, device)
                d_grads.append((gp, gn))
            torch.cuda.synchronize()
            # outputs are read back after every step's main work, while later mini-batches are already in flight
            p.start(*d_batches[0], more=d_batches[1:lookahead])
            for i in range(steps):
                nxt = d_batches[i + lookahead] if i + lookahead < steps else None
                st = p.sets[p.step(d_grads[i][0], d_grads[i][1], lr, next_batch=nxt)]
                perm_o, n_pop_o, L_pop, L_non, n_cold_o, pooled_pop_o, pooled_non_o = expect[i]
                p.main.synchronize()
                assert st.counts.cpu().tolist() == [n_pop_o, B - n_pop_o, L_pop, L_non], ("counts", i)
                assert np.array_equal(st.perm[:B].cpu().numpy(), perm_o), ("perm", i)
                assert int(st.n_cold.item()) == n_cold_o, ("n_cold", i, int(st.n_cold.item()), n_cold_o)
                bags_pop, bags_non = T * n_pop_o * S, T * (B - n_pop_o) * S
                assert np.array_equal(st.pooled_pop[:bags_pop].cpu().numpy(), pooled_pop_o), ("pooled_pop", i)
                assert np.array_equal(st.pooled_non[:bags_non].cpu().numpy(), pooled_non_o), ("pooled_non", i)
            p.drain()
            p.status()
        assert np.array_equal(p.cache[:n_hot].cpu().numpy(), cache_o[:n_hot]), "hot cache"
        host = table.numpy()
        assert np.array_equal(host[staged_rows], np.asarray(table_o[staged_rows])), "written-back host rows"
        assert not np.array_equal(np.asarray(table_o[staged_rows]), rows_of(staged_rows)), "the updates changed nothing"
        far = rng.integers(0, N, 4096)
        far = far[~np.isin(far, staged_rows)]
        assert np.array_equal(host[far], rows_of(far)), "host rows nobody touched"
        stats = dict(N=N, batch=B, steps=steps, n_hot=n_hot, n_pop=[e[1] for e in expect], n_cold=[e[4] for e in expect],
                     shared_cold_rows=shared, staged_rows=len(staged_rows))
        if verbose:
            print(f"[{spec.name} full size, hl_pipe] {stats}")
        return stats
    finally:
        if p is not None:
            p.close()
        torch.cuda.synchronize()
        hl.hl_host_free(table.data_ptr())
        del table_o
        tmp.cleanup()


def run_recalibration_check(spec, steps_per_phase: int = 2, device: str = "cuda:0"):
    """Learning phase, some mini-batches, flush of the popular rows, a second learning phase over a later window of
    mini-batches (another popular set), more mini-batches, flush: after each flush the host table must equal the
    oracle's table.  Integer data, so every comparison is exact."""
    import paper_2204_05436_b200 as hl

    if isinstance(spec, str):
        spec = gen.CONFIGS[spec]
    geom = gen.make_geometry(spec)
    T, D, S, B = geom.num_tables, geom.dim, geom.bags_per_sample, spec.batch
    N, n_bags, P, lr = geom.total_rows, T * B * S, spec.profile_batches, 0.125
    max_nnz = max_nnz_of(spec, geom, B)
    K = orc.hot_capacity(spec.hot_policy, N, D)
    hot_cap, staging_cap = max(1, min(K, N)), max(1, min(N, max_nnz))
    table_o = gen.table_values(np.arange(N), D, spec.seed, integer=True)
    host_table = torch.from_numpy(table_o.copy()).pin_memory()
    h = hl.Hotline(geom.table_rows, D, S, B, max_nnz, hot_cap, staging_cap, host_table, device=device)
    pol, p_num, p_den = policy_args(spec.hot_policy)
    hot_sets = []
    try:
        with torch.cuda.stream(h.main):
            next_batch = 0
            for phase in range(2):
                # learning phase over the next P mini-batches, scaled differently per phase so the sets differ
                prof = [gen.make_batch(spec, geom, next_batch + i) for i in range(P if phase == 0 else max(1, P // 3))]
                next_batch += len(prof)
                cnt = orc.access_counts([(b.indices, b.offsets) for b in prof], B, geom.table_rows, S)
                hot_o = orc.select_hot(cnt, min(K, hot_cap))
                hot_sets.append(hot_o)
                remap_o = orc.build_remap(hot_o, N)
                cache_o = np.zeros((hot_cap + staging_cap, D), dtype=np.float32)
                cache_o[:len(hot_o)] = orc.load_hot_cache(table_o, hot_o)
                for i, b in enumerate(prof):
                    h.profile(_t(b.indices, device), _t(b.offsets, device), B, reset=(i == 0))
                h.profile(None, None, finalize=True, policy=pol, p_num=p_num, p_den=p_den)
                h.build_remap(load_rows=True)
                h.status()
                assert np.array_equal(h.hot_rows[:len(hot_o)].cpu().numpy(), hot_o.astype(np.int32)), ("hot", phase)
                for step in range(steps_per_phase):
                    batch = gen.make_batch(spec, geom, next_batch)
                    grad_full = gen.grad_values(spec.seed, next_batch, 2, n_bags, D, integer=True)
                    next_batch += 1
                    perm_o, n_pop_o, _, _, _ = orc.fragment(batch.indices, batch.offsets, B, geom.table_rows, remap_o, S)
                    g_pop, _ = mu_grad(grad_full, perm_o[:n_pop_o], T, B, S)
                    g_non, _ = mu_grad(grad_full, perm_o[n_pop_o:], T, B, S)
                    orc.hotline_step(table_o, cache_o, hot_cap, remap_o, batch.indices, batch.offsets, B,
                                     geom.table_rows, S, g_pop, g_non, lr)
                    gp = torch.zeros((n_bags, D), dtype=torch.float32, device=device)
                    gn = torch.zeros((n_bags, D), dtype=torch.float32, device=device)
                    gp[:len(g_pop)] = _t(g_pop, device)
                    gn[:len(g_non)] = _t(g_non, device)
                    h.step(_t(batch.indices, device), _t(batch.offsets, device), B, gp, gn, lr)
                    h.status()
                orc.flush_hot(table_o, cache_o, hot_o)
                h.flush_hot()
                h.status()
                assert np.array_equal(h.host_table.numpy(), table_o), ("host table after flush", phase)
    finally:
        h.close()
    return dict(hot_sets_differ=not np.array_equal(hot_sets[0], hot_sets[1]), n_hot=[len(x) for x in hot_sets])
