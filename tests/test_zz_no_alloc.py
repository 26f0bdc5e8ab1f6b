"""The allocation-free backward entry point (hl_embbag_bwd_sgd_static) against the regular one.

Some users of the library cannot allocate device memory at all (a plug-in inside an application that owns the
GPU's memory, a loop that must stay out of the allocator), so they cannot give the library a workspace.  For them
the library carries a fixed scratch array in its own image.  This test calls that entry point through the C
boundary twice in a row, with different shapes, and checks each result against hl_embbag_bwd_sgd on the same
inputs (and against the CPU oracle).  The second call finds the first call's data still in the array, which is the
case the entry point has to cope with; the test creates every buffer and context it uses, so it does not depend on
what ran before it.
"""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu

RTOL, ATOL = 1e-5, 1e-6


def _case(seed, n_bags, cache_rows, dim, max_pool):
    rng = np.random.default_rng(seed)
    sizes = rng.integers(0, max_pool + 1, n_bags)
    offsets = np.concatenate([[0], np.cumsum(sizes)]).astype(np.int32)
    # a skewed id distribution gives long runs of equal ids as well as singletons
    ids = np.minimum((rng.pareto(1.1, int(offsets[-1])) * 3).astype(np.int64), cache_rows - 1).astype(np.int32)
    cache = rng.standard_normal((cache_rows, dim)).astype(np.float32)
    grad = rng.standard_normal((n_bags, dim)).astype(np.float32)
    return offsets, ids, cache, grad


def _run_regular(hl, offsets, ids, cache, grad, lr, dev):
    """hl_embbag_bwd_sgd with a context over a caller-allocated workspace."""
    n_bags, nnz, (rows, dim) = len(offsets) - 1, len(ids), cache.shape
    geom = hl.make_geometry([rows], dim, 1)
    ws_bytes = hl.hl_workspace_bytes(geom, n_bags, nnz, rows, 0)
    ws = torch.empty(ws_bytes, dtype=torch.uint8, device=dev)
    ctx = hl.hl_create(geom, n_bags, nnz, rows, 0, ws, ws_bytes)
    try:
        d_cache = torch.from_numpy(cache.copy()).to(dev)
        d_off, d_ids = torch.from_numpy(offsets).to(dev), torch.from_numpy(ids).to(dev)
        d_grad = torch.from_numpy(grad).to(dev)
        d_n = torch.tensor([n_bags], dtype=torch.int32, device=dev)
        torch.cuda.synchronize()
        ub = hl.make_ubatch(d_off, d_ids, nnz)
        hl.hl_embbag_bwd_sgd(ctx, d_cache, ub, d_n, d_grad, lr, torch.cuda.current_stream().cuda_stream)
        hl.hl_status(ctx)
        return d_cache.cpu().numpy()
    finally:
        torch.cuda.synchronize()
        hl.hl_destroy(ctx)


def _run_static(hl, offsets, ids, cache, grad, lr, dev):
    n_bags, nnz, (rows, dim) = len(offsets) - 1, len(ids), cache.shape
    d_cache = torch.from_numpy(cache.copy()).to(dev)
    d_off, d_ids = torch.from_numpy(offsets).to(dev), torch.from_numpy(ids).to(dev)
    d_grad = torch.from_numpy(grad).to(dev)
    d_status = torch.full((1,), 77, dtype=torch.int32, device=dev)
    torch.cuda.synchronize()
    hl.hl_embbag_bwd_sgd_static(d_cache, rows, dim, d_off, d_ids, n_bags, nnz, d_grad, lr, d_status,
                                torch.cuda.current_stream().cuda_stream)
    torch.cuda.synchronize()
    assert int(d_status.item()) == 0
    return d_cache.cpu().numpy()


def test_static_backward_matches_the_regular_entry_point_twice_in_a_row():
    import paper_2204_05436_b200 as hl
    from oracle import hotline_oracle as orc
    dev = "cuda:0"
    torch.cuda.set_device(0)
    # second call: fewer lookups, wider rows, other ids -- the array still holds the first call's data
    for seed, n_bags, rows, dim, pool in [(1, 6000, 4000, 32, 9), (2, 1500, 900, 128, 4)]:
        offsets, ids, cache, grad = _case(seed, n_bags, rows, dim, pool)
        assert len(ids) <= hl.HL_STATIC_MAX_NNZ
        want = _run_regular(hl, offsets, ids, cache, grad, 0.05, dev)
        got = _run_static(hl, offsets, ids, cache, grad, 0.05, dev)
        np.testing.assert_allclose(got, want, rtol=RTOL, atol=ATOL)
        ref = cache.copy()
        orc.embbag_bwd_sgd(ref, ids, offsets, grad, 0.05)
        np.testing.assert_allclose(got, ref, rtol=RTOL, atol=ATOL)
        assert not np.array_equal(got, cache)


def test_static_backward_refuses_sizes_beyond_its_array():
    import paper_2204_05436_b200 as hl
    dev = "cuda:0"
    d = torch.zeros(16, dtype=torch.float32, device=dev)
    i = torch.zeros(16, dtype=torch.int32, device=dev)
    s = torch.cuda.current_stream().cuda_stream
    with pytest.raises(hl.HotlineError) as e:
        hl.hl_embbag_bwd_sgd_static(d, 4, 4, i, i, 4, hl.HL_STATIC_MAX_NNZ + 1, d, 0.1, None, s)
    assert e.value.status == hl.HL_ECAPACITY
    with pytest.raises(hl.HotlineError) as e:
        hl.hl_embbag_bwd_sgd_static(d, 4, hl.HL_STATIC_MAX_DIM + 4, i, i, 4, 4, d, 0.1, None, s)
    assert e.value.status == hl.HL_ECAPACITY
