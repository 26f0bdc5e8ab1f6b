"""The wide-id index path (hl_wide_*: 64-bit global row ids, hashed counter, hashed remap) against the oracle: on a
small model, where the rest of the path then runs on its slots and the results must equal the oracle's step, and on a
model with more than 2^31 rows, where only the index-only calls run (no table of that size is allocated)."""
import numpy as np
import pytest
import torch

import gen
from oracle import hotline_oracle as orc

pytestmark = pytest.mark.gpu

DEV = "cuda:0"
RTOL, ATOL = 1e-5, 1e-6


def _t(x):
    return torch.from_numpy(np.ascontiguousarray(x)).to(DEV)


class _Wide:
    """Buffers and context of the wide-id calls for one geometry."""

    def __init__(self, hl, table_rows, S, B, max_nnz, hot_cap, staging_cap, counter_slots):
        self.hl, self.T, self.S, self.B = hl, len(table_rows), S, B
        self.hot_cap, self.max_nnz = hot_cap, max_nnz
        self.geom = hl.make_geometry(table_rows, 4, S)
        ws_bytes = hl.hl_wide_workspace_bytes(self.geom, B, max_nnz, hot_cap, staging_cap, counter_slots)
        self.ws = torch.empty(ws_bytes, dtype=torch.uint8, device=DEV)
        self.w = hl.hl_wide_create(self.geom, B, max_nnz, hot_cap, staging_cap, counter_slots, self.ws, ws_bytes)
        i32, i64 = torch.int32, torch.int64
        n_bags = self.T * B * S
        z = lambda n, dt: torch.zeros(max(1, n), dtype=dt, device=DEV)   # noqa: E731
        self.hot_rows, self.n_hot = z(hot_cap, i64), z(1, i64)
        self.perm, self.counts = z(B, i32), z(4, i32)
        self.pop_off, self.pop_ids = z(n_bags + 1, i32), z(max_nnz, i32)
        self.non_off, self.non_rows, self.non_slots = z(n_bags + 1, i32), z(max_nnz, i64), z(max_nnz, i32)
        self.cold_rows, self.n_cold = z(staging_cap, i64), z(1, i64)
        self.pop = hl.make_ubatch(self.pop_off, self.pop_ids, max_nnz)
        self.stream = torch.cuda.current_stream().cuda_stream

    def close(self):
        torch.cuda.synchronize()
        self.hl.hl_wide_destroy(self.w)

    def learn(self, batches, policy, p_num, p_den, row_bytes):
        hl = self.hl
        for i, b in enumerate(batches):
            hb = hl.make_batch(_t(b.indices), _t(b.offsets), self.B, len(b.indices))
            hl.hl_wide_profile_hot(self.w, hb, i == 0, False, 0, 0, 1, row_bytes, self.hot_rows, self.n_hot, self.stream)
            torch.cuda.synchronize()
        hl.hl_wide_profile_hot(self.w, None, False, True, policy, p_num, p_den, row_bytes, self.hot_rows, self.n_hot,
                               self.stream)
        hl.hl_wide_build_remap(self.w, self.hot_rows, self.n_hot, self.stream)
        assert hl.hl_wide_status(self.w) == hl.HL_OK
        return self.hot_rows[:int(self.n_hot.item())].cpu().numpy()

    def index(self, b):
        hl = self.hl
        d_idx, d_off = _t(b.indices), _t(b.offsets)
        hb = hl.make_batch(d_idx, d_off, self.B, len(b.indices))
        hl.hl_wide_fragment(self.w, hb, self.perm, self.counts, self.pop, self.non_off, self.non_rows, self.max_nnz,
                            self.stream)
        hl.hl_wide_index_cold(self.w, self.non_off, self.non_rows, self.max_nnz, self.counts[1:], self.non_slots,
                              self.cold_rows, self.n_cold, self.stream)
        assert hl.hl_wide_status(self.w) == hl.HL_OK


def _check_index(wd, b, table_rows, S, remap, hot_cap):
    """perm, counts, both CSRs, X's global rows, the cold rows and the unified slots, bit for bit."""
    B = wd.B
    perm, n_pop, O, X, _ = orc.fragment(b.indices, b.offsets, B, table_rows, remap, S)
    C, x_slots = orc.gather_cold(X.ids, remap, hot_cap)
    assert wd.counts.cpu().tolist() == [n_pop, B - n_pop, len(O.ids), len(X.ids)]
    assert np.array_equal(wd.perm[:B].cpu().numpy(), perm)
    assert np.array_equal(wd.pop_off[:len(O.offsets)].cpu().numpy(), O.offsets)
    assert np.array_equal(wd.pop_ids[:len(O.ids)].cpu().numpy(), O.ids)
    assert np.array_equal(wd.non_off[:len(X.offsets)].cpu().numpy(), X.offsets)
    assert int(wd.n_cold.item()) == len(C)
    assert np.array_equal(wd.cold_rows[:len(C)].cpu().numpy(), C)
    assert np.array_equal(wd.non_slots[:len(x_slots)].cpu().numpy(), x_slots)
    return perm, n_pop, O, X, C, x_slots


def test_small_model_index_calls_and_the_rest_of_the_path_on_their_slots():
    """Ragged tables, multi-hot bags: the hashed structures give the oracle's hot set, fragments, cold rows and
    slots; forward, update and write-back then run through an ordinary context on those slots and must equal the
    oracle's step (integer data: bit for bit)."""
    import paper_2204_05436_b200 as hl
    spec = gen.WorkloadSpec(name="wide_small", num_tables=7, dim=16, batch=600, rows=("loguniform", 20, 40_000, 5),
                            alpha=tuple([1.15] * 7), pooling=("poisson", 3.0, 8), hot_policy=("fraction", 8, 100),
                            profile_batches=5, seed=31)
    geom = gen.make_geometry(spec)
    T, D, S, B, N = geom.num_tables, geom.dim, 1, spec.batch, geom.total_rows
    max_nnz = T * B * 8
    K = orc.hot_capacity(spec.hot_policy, N, D)
    prof = [gen.make_batch(spec, geom, i) for i in range(spec.profile_batches)]
    cnt = orc.access_counts([(b.indices, b.offsets) for b in prof], B, geom.table_rows, S)
    hot_o = orc.select_hot(cnt, K)
    remap = orc.build_remap(hot_o, N)
    wd = _Wide(hl, geom.table_rows, S, B, max_nnz, K, max_nnz, counter_slots=4 * len(np.flatnonzero(cnt)))
    table0 = gen.table_values(np.arange(N), D, spec.seed, integer=True)
    host_table = torch.from_numpy(table0.copy()).pin_memory()
    h = hl.Hotline(geom.table_rows, D, S, B, max_nnz, K, max_nnz, host_table, device=DEV)
    try:
        hot_g = wd.learn(prof, hl.HL_HOT_FRACTION_ROWS, 8, 100, 4 * D)
        assert np.array_equal(hot_g, hot_o)
        # minimum-share policy through the same counter
        hl.hl_wide_profile_hot(wd.w, None, False, True, hl.HL_HOT_MIN_SHARE, 1, 3000, 4 * D, wd.hot_rows, wd.n_hot,
                               wd.stream)
        torch.cuda.synchronize()
        want = orc.select_hot(cnt, K, (1, 3000))
        assert np.array_equal(wd.hot_rows[:int(wd.n_hot.item())].cpu().numpy(), want)
        hot_g = wd.learn(prof, hl.HL_HOT_FRACTION_ROWS, 8, 100, 4 * D)

        with torch.cuda.stream(h.main):
            h.set_hot_rows(_t(hot_o))
            h.build_remap(load_rows=True)
            h.status()
        torch.cuda.synchronize()
        table_o = table0.copy()
        cache_o = np.zeros((K + max_nnz, D), dtype=np.float32)
        cache_o[:len(hot_o)] = orc.load_hot_cache(table0, hot_o)
        n_bags = T * B * S
        for step in range(3):
            b = gen.make_batch(spec, geom, spec.profile_batches + step)
            wd.index(b)
            perm, n_pop, O, X, C, x_slots = _check_index(wd, b, geom.table_rows, S, remap, K)
            assert np.array_equal(wd.non_rows[:len(X.ids)].cpu().numpy(), X.ids.astype(np.int64))
            grad = gen.grad_values(spec.seed, step, 2, n_bags, D, integer=True)
            src = lambda smp: ((np.arange(T)[:, None] * B + np.asarray(smp, dtype=np.int64)[None, :])).reshape(-1)  # noqa: E731
            g_pop, g_non = grad[src(perm[:n_pop])], grad[src(perm[n_pop:])]
            out = orc.hotline_step(table_o, cache_o, K, remap, b.indices, b.offsets, B, geom.table_rows, S, g_pop, g_non,
                                   0.125)
            # the rest of the path on the wide calls' slots, through the ordinary context
            s = wd.stream
            cold32 = wd.cold_rows.to(torch.int32)
            non = hl.make_ubatch(wd.non_off, wd.non_slots, max_nnz)
            pooled_pop = torch.zeros((n_bags, D), device=DEV)
            pooled_non = torch.zeros((n_bags, D), device=DEV)
            gp, gn = torch.zeros((n_bags, D), device=DEV), torch.zeros((n_bags, D), device=DEV)
            gp[:len(g_pop)], gn[:len(g_non)] = _t(g_pop), _t(g_non)
            torch.cuda.synchronize()
            hl.hl_stage_cold(h.ctx, h.host_table, h.cache, 0, max_nnz, cold32, wd.n_cold, None, s)
            hl.hl_embbag_fwd(h.ctx, h.cache, wd.pop, wd.counts, pooled_pop, s)
            hl.hl_embbag_bwd_sgd(h.ctx, h.cache, wd.pop, wd.counts, gp, 0.125, s)
            hl.hl_embbag_fwd(h.ctx, h.cache, non, wd.counts[1:], pooled_non, s)
            hl.hl_embbag_bwd_sgd(h.ctx, h.cache, non, wd.counts[1:], gn, 0.125, s)
            hl.hl_scatter_cold_at(h.ctx, h.cache, 0, max_nnz, cold32, wd.n_cold, h.host_table, s)
            assert h.status() == hl.HL_OK
            assert np.array_equal(pooled_pop[:len(out[5])].cpu().numpy(), out[5])
            assert np.array_equal(pooled_non[:len(out[6])].cpu().numpy(), out[6])
            assert np.array_equal(h.cache[:len(hot_o)].cpu().numpy(), cache_o[:len(hot_o)])
            assert np.array_equal(h.host_table.numpy(), table_o)
    finally:
        wd.close()
        h.close()


def _mem_available_gib():
    for line in open("/proc/meminfo"):
        if line.startswith("MemAvailable"):
            return int(line.split()[1]) / 2 ** 20
    return 0.0


def test_index_calls_on_a_model_with_more_than_2_to_31_rows():
    """Four tables with 2.2 billion rows together (the second one starts beyond 2^31 - 1): hot set, fragments, cold
    rows and slots against the oracle, which works on 64-bit ids throughout.  No table is allocated."""
    import paper_2204_05436_b200 as hl
    if _mem_available_gib() < 96:
        pytest.skip("the oracle's dense arrays over 2.2 billion rows need about 50 GB of host memory")
    spec = gen.WorkloadSpec(name="wide_large", num_tables=4, dim=16, batch=2048,
                            rows=("list", (1_500_000_000, 700_000_000, 5_000_000, 300)), alpha=(1.1, 1.2, 1.05, 1.3),
                            hot_policy=("topk", 6000), profile_batches=4, seed=37)
    geom = gen.make_geometry(spec)
    T, S, B, N = geom.num_tables, 1, spec.batch, geom.total_rows
    assert N > 2 ** 31 and geom.base[1] > 2 ** 30
    K = 6000
    prof = [gen.make_batch(spec, geom, i) for i in range(spec.profile_batches)]
    cnt = orc.access_counts([(b.indices, b.offsets) for b in prof], B, geom.table_rows, S)
    hot_o = orc.select_hot(cnt, K)
    del cnt
    assert hot_o.max() > 2 ** 31
    remap = orc.build_remap(hot_o, N)
    max_nnz = T * B
    wd = _Wide(hl, geom.table_rows, S, B, max_nnz, K, max_nnz, counter_slots=1 << 16)
    try:
        hot_g = wd.learn(prof, hl.HL_HOT_TOPK_ROWS, K, 1, 64)
        assert hot_g.dtype == np.int64 and np.array_equal(hot_g, hot_o)
        for step in range(2):
            b = gen.make_batch(spec, geom, spec.profile_batches + step)
            wd.index(b)
            _, _, _, X, C, _ = _check_index(wd, b, geom.table_rows, S, remap, K)
            assert len(C) > 0 and C.max() > 2 ** 31 and X.ids.dtype == np.int64
            assert np.array_equal(wd.non_rows[:len(X.ids)].cpu().numpy(), X.ids)
    finally:
        wd.close()
