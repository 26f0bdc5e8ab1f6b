"""Error paths on the device that must end in a status word, never in a hang or a fault: the bounded waits of the
chained scan, of the chained sort passes and of the row movers are made to run out (a participant withholds what
the others wait for, and the poll limit is lowered so that they give up within microseconds), and skipped lookups
(negative ids) go through the combined backward sort.  After every such call the same context must work normally.
"""
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


def _tiny_hotline(hl):
    spec = gen.CONFIGS["tiny"]
    geom = gen.make_geometry(spec)
    N, D, B = geom.total_rows, spec.dim, spec.batch
    table0 = gen.table_values(np.arange(N), D, spec.seed)
    host_table = torch.from_numpy(table0.copy()).pin_memory()
    n_bags = geom.num_tables * B
    h = hl.Hotline(geom.table_rows, D, 1, B, n_bags, 4000, n_bags, host_table, device=DEV)
    return spec, geom, table0, h


def test_scan_wait_runs_out_and_the_context_recovers():
    """hl_fragment's scan over 8,192 destination bags has five tiles; tile 1 publishes nothing, so the tiles behind
    it poll 200 times and give up: HL_ETIMEOUT, no hang.  The next hl_fragment on the same context is exact."""
    import paper_2204_05436_b200 as hl
    spec, geom, table0, h = _tiny_hotline(hl)
    try:
        with torch.cuda.stream(h.main):
            rng = np.random.default_rng(5)
            hot = np.sort(rng.choice(geom.total_rows, 3000, replace=False)).astype(np.int64)
            h.set_hot_rows(_t(hot))
            h.build_remap(load_rows=True)
            assert h.status() == hl.HL_OK
            b = gen.make_batch(spec, geom, 3)
            d_idx, d_off = _t(b.indices), _t(b.offsets)
            hl.hl_test_bounded_waits(h.ctx, 200, 1)
            h.fragment(d_idx, d_off, spec.batch)
            assert h.status(raise_on_error=False) == hl.HL_ETIMEOUT
            hl.hl_test_bounded_waits(h.ctx, 0, -1)
            h.fragment(d_idx, d_off, spec.batch)
            assert h.status() == hl.HL_OK
            remap = orc.build_remap(hot, geom.total_rows)
            perm, n_pop, O, X, _ = orc.fragment(b.indices, b.offsets, spec.batch, geom.table_rows, remap, 1)
            assert h.counts.cpu().tolist() == [n_pop, spec.batch - n_pop, len(O.ids), len(X.ids)]
            assert np.array_equal(h.perm[:spec.batch].cpu().numpy(), perm)
            assert np.array_equal(h.pop_ids[:len(O.ids)].cpu().numpy(), O.ids)
            assert np.array_equal(h.non_ids[:len(X.ids)].cpu().numpy(), X.ids)
            assert np.array_equal(h.non_offsets[:len(X.offsets)].cpu().numpy(), X.offsets)
    finally:
        h.close()


def test_sort_wait_runs_out_and_the_context_recovers():
    """The backward's sort of 8,192 (slot, bag) pairs has four tiles per pass; tile 1 publishes nothing.  The call
    returns with HL_ETIMEOUT; afterwards hl_embbag_bwd_sgd on the same context matches the oracle."""
    import paper_2204_05436_b200 as hl
    rng = np.random.default_rng(9)
    rows, dim, n_bags = 5000, 16, 8192
    ids = np.minimum((rng.pareto(1.2, n_bags) * 40).astype(np.int64), rows - 1).astype(np.int32)
    offsets = np.arange(n_bags + 1, dtype=np.int32)
    cache = rng.standard_normal((rows, dim)).astype(np.float32)
    grad = rng.standard_normal((n_bags, dim)).astype(np.float32)
    geom = hl.make_geometry([rows], dim, 1)
    ws_bytes = hl.hl_workspace_bytes(geom, n_bags, n_bags, rows, 0)
    ws = torch.empty(ws_bytes, dtype=torch.uint8, device=DEV)
    ctx = hl.hl_create(geom, n_bags, n_bags, rows, 0, ws, ws_bytes)
    try:
        d_cache, d_off, d_ids, d_grad = _t(cache), _t(offsets), _t(ids), _t(grad)
        d_n = torch.tensor([n_bags], dtype=torch.int32, device=DEV)
        sk, sb = (torch.zeros(n_bags, dtype=torch.int32, device=DEV) for _ in range(2))
        sn = torch.zeros(4, dtype=torch.int32, device=DEV)
        ub = hl.make_ubatch(d_off, d_ids, n_bags)
        stream = torch.cuda.current_stream().cuda_stream
        torch.cuda.synchronize()
        hl.hl_test_bounded_waits(ctx, 200, 1)
        hl.hl_embbag_bwd_prepare(ctx, ub, d_n, sk, sb, sn, stream)
        assert hl.hl_status(ctx, raise_on_error=False) == hl.HL_ETIMEOUT
        hl.hl_test_bounded_waits(ctx, 0, -1)
        hl.hl_embbag_bwd_sgd(ctx, d_cache, ub, d_n, d_grad, 0.05, stream)
        assert hl.hl_status(ctx) == hl.HL_OK
        want = cache.copy()
        orc.embbag_bwd_sgd(want, ids, offsets, grad, 0.05)
        np.testing.assert_allclose(d_cache.cpu().numpy(), want, rtol=RTOL, atol=ATOL)
    finally:
        torch.cuda.synchronize()
        hl.hl_destroy(ctx)


def test_mover_wait_runs_out_and_the_context_recovers():
    """The first stage of the row mover's first CTA issues no copies, so the bytes its barrier expects never arrive:
    that CTA gives up after 200 polls, leaves its rows unmoved and returns; the others finish.  HL_ETIMEOUT, and
    the next load of the hot cache on the same context is a bit copy of the table's rows."""
    import paper_2204_05436_b200 as hl
    spec, geom, table0, h = _tiny_hotline(hl)
    try:
        with torch.cuda.stream(h.main):
            hot = np.arange(0, 4000 * 20, 20, dtype=np.int64)
            h.set_hot_rows(_t(hot))
            hl.hl_test_bounded_waits(h.ctx, 200, 0)
            h.build_remap(load_rows=True)
            assert h.status(raise_on_error=False) == hl.HL_ETIMEOUT
            hl.hl_test_bounded_waits(h.ctx, 0, -1)
            h.cache.zero_()
            h.build_remap(load_rows=True)
            assert h.status() == hl.HL_OK
            assert np.array_equal(h.cache[:len(hot)].cpu().numpy().view(np.uint32), table0[hot].view(np.uint32))
    finally:
        h.close()


def test_combined_backward_sort_keeps_skipped_lookups_of_the_popular_block_apart():
    """hl_embbag_bwd_prepare2 / apply2 with negative (skipped) ids among O's lookups: they sort to the end of O's
    block and must not displace any of X's pairs, so both updates equal the oracle's on the remaining lookups."""
    import paper_2204_05436_b200 as hl
    rng = np.random.default_rng(17)
    T, D, B = 3, 8, 700
    hot_cap, staging = 900, 300
    rows = hot_cap + staging
    n_pop, n_non = 450, 250
    geom = hl.make_geometry([2000] * T, D, 1)
    max_nnz = T * B * 3
    ws_bytes = hl.hl_workspace_bytes(geom, B, max_nnz, hot_cap, staging)
    ws = torch.empty(ws_bytes, dtype=torch.uint8, device=DEV)
    ctx = hl.hl_create(geom, B, max_nnz, hot_cap, staging, ws, ws_bytes)

    def csr(n_samples, hi):
        sizes = rng.integers(0, 4, T * n_samples)
        off = np.concatenate([[0], np.cumsum(sizes)]).astype(np.int32)
        ids = np.minimum((rng.pareto(1.1, int(off[-1])) * 5).astype(np.int64), hi - 1).astype(np.int32)
        return off, ids

    try:
        o_off, o_ids = csr(n_pop, hot_cap)
        x_off, x_ids = csr(n_non, rows)
        skipped = rng.choice(len(o_ids), 37, replace=False)
        o_ids[skipped] = -1
        x_ids[rng.choice(len(x_ids), 5, replace=False)] = -1
        cache = rng.standard_normal((rows, D)).astype(np.float32)
        g_pop = rng.standard_normal((T * n_pop, D)).astype(np.float32)
        g_non = rng.standard_normal((T * n_non, D)).astype(np.float32)

        def padded(a, n):
            out = np.zeros(n, dtype=a.dtype)
            out[:len(a)] = a
            return out

        d_counts = torch.tensor([n_pop, n_non], dtype=torch.int32, device=DEV)
        sk, sb = (torch.zeros(max_nnz, dtype=torch.int32, device=DEV) for _ in range(2))
        sn = torch.zeros(4, dtype=torch.int32, device=DEV)
        d_cache, d_gp, d_gn = _t(cache), _t(g_pop), _t(g_non)
        stream = torch.cuda.current_stream().cuda_stream
        # the device tensors behind the two micro-batches must stay alive while the calls run
        o_t = (_t(padded(o_off, T * B + 1)), _t(padded(o_ids, max_nnz)))
        x_t = (_t(padded(x_off, T * B + 1)), _t(padded(x_ids, max_nnz)))
        d_o, d_x = hl.make_ubatch(o_t[0], o_t[1], max_nnz), hl.make_ubatch(x_t[0], x_t[1], max_nnz)
        torch.cuda.synchronize()
        hl.hl_embbag_bwd_prepare2(ctx, d_o, d_counts, d_x, d_counts[1:], sk, sb, sn, stream)
        hl.hl_embbag_bwd_apply2(ctx, d_cache, sk, sb, sn, 0, d_gp, 0.05, stream)
        hl.hl_embbag_bwd_apply2(ctx, d_cache, sk, sb, sn, 1, d_gn, 0.05, stream)
        assert hl.hl_status(ctx) == hl.HL_OK
        assert sn.cpu().tolist()[:3] == [len(o_ids), len(x_ids), len(o_ids) + len(x_ids)]

        def drop_skipped(off, ids):
            bag = np.repeat(np.arange(len(off) - 1), np.diff(off))
            ok = ids >= 0
            new_off = np.concatenate([[0], np.cumsum(np.bincount(bag[ok], minlength=len(off) - 1))]).astype(np.int32)
            return new_off, ids[ok]

        want = cache.copy()
        orc.embbag_bwd_sgd(want, *drop_skipped(o_off, o_ids)[::-1], g_pop, 0.05)
        orc.embbag_bwd_sgd(want, *drop_skipped(x_off, x_ids)[::-1], g_non, 0.05)
        np.testing.assert_allclose(d_cache.cpu().numpy(), want, rtol=RTOL, atol=ATOL)
    finally:
        torch.cuda.synchronize()
        hl.hl_destroy(ctx)
