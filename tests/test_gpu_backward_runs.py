"""The backward call on slot lists built to hit every border case of its chunking.

hl_embbag_bwd_sgd sorts the (slot, bag) pairs, cuts the sorted list into chunks of 32 lookups and sums each run of
equal slots: inside a chunk, over two neighbouring chunks (the group of the first chunk reads on into the second, whose
group leaves those lookups alone), or, for longer runs, through partial sums that a second kernel adds up.  The cases
here fix the run lengths and where the runs start, so that runs end exactly at a chunk's last lookup, start at its
first, cover one, two, three or many chunks exactly or with one lookup more or less, follow one another without a gap,
and end the list in a ragged chunk.  Data are integers (every sum exact), so the updated rows must equal the oracle's
bit for bit, for every row width class of the kernels.
"""
import numpy as np
import pytest
import torch

from oracle import hotline_oracle as orc

pytestmark = pytest.mark.gpu

DEV = "cuda:0"

# run lengths, in the order of their slots; each list is laid out from position 0 of the sorted list
CASES = {
    "borders": [32, 1, 31, 33, 31, 1, 63, 1, 64, 65, 95, 96, 97, 5],
    "two_chunk_runs": [20, 24, 24, 24, 24, 24, 24, 24, 24, 24, 24, 12, 40, 40, 40, 7],
    "from_first_lookup": [32, 32, 64, 32, 96, 32, 33, 31, 32],
    "one_long_run": [3, 1000, 2],
    "long_then_short": [31, 2, 200, 1, 1, 1, 62, 2, 62, 3],
    "singles": [1] * 70,
    "all_one_row": [517],
    "ragged_end": [30, 3, 64, 10],
}


def _lookups(lengths, seed):
    """One lookup per bag; slot of run r is 3 * r + 1 (gaps between the slots that are used); bags in random order, so
    that the sort has work to do and a run's gradient rows are scattered."""
    rng = np.random.default_rng(seed)
    ids = np.concatenate([np.full(n, 3 * r + 1, dtype=np.int32) for r, n in enumerate(lengths)])
    rng.shuffle(ids)
    n_bags = len(ids)
    offsets = np.arange(n_bags + 1, dtype=np.int32)
    return ids, offsets, 3 * len(lengths) + 2


def _backward(hl, ids, offsets, cache, grad, lr):
    n_bags, nnz, (rows, dim) = len(offsets) - 1, len(ids), cache.shape
    geom = hl.make_geometry([rows], dim, 1)
    ws_bytes = hl.hl_workspace_bytes(geom, n_bags, nnz, rows, 0)
    ws = torch.empty(ws_bytes, dtype=torch.uint8, device=DEV)
    ctx = hl.hl_create(geom, n_bags, nnz, rows, 0, ws, ws_bytes)
    try:
        d_cache = torch.from_numpy(cache.copy()).to(DEV)
        d_off, d_ids = torch.from_numpy(offsets).to(DEV), torch.from_numpy(ids).to(DEV)
        d_grad = torch.from_numpy(grad).to(DEV)
        d_n = torch.tensor([n_bags], dtype=torch.int32, device=DEV)
        ub = hl.make_ubatch(d_off, d_ids, nnz)
        stream = torch.cuda.current_stream().cuda_stream
        hl.hl_embbag_bwd_sgd(ctx, d_cache, ub, d_n, d_grad, lr, stream)
        hl.hl_status(ctx)
        once = d_cache.cpu().numpy()
        hl.hl_embbag_bwd_sgd(ctx, d_cache, ub, d_n, d_grad, lr, stream)      # the call leaves its scratch reusable
        hl.hl_status(ctx)
        return once, d_cache.cpu().numpy()
    finally:
        torch.cuda.synchronize()
        hl.hl_destroy(ctx)


@pytest.mark.parametrize("dim", [16, 32, 64, 128, 200, 512])
@pytest.mark.parametrize("case", sorted(CASES))
def test_backward_on_runs_that_hit_the_chunk_borders(case, dim):
    import paper_2204_05436_b200 as hl
    ids, offsets, rows = _lookups(CASES[case], seed=len(case) + dim)
    rng = np.random.default_rng(dim)
    cache = rng.integers(-8, 9, (rows, dim)).astype(np.float32)
    grad = rng.integers(-4, 5, (len(ids), dim)).astype(np.float32)
    lr = 0.5                                     # integers times a power of two: every update is exact
    want1 = cache.copy()
    orc.embbag_bwd_sgd(want1, ids, offsets, grad, lr)
    want2 = want1.copy()
    orc.embbag_bwd_sgd(want2, ids, offsets, grad, lr)
    got1, got2 = _backward(hl, ids, offsets, cache, grad, lr)
    assert np.array_equal(got1, want1), f"{case}, dim {dim}: {int((got1 != want1).any(axis=1).sum())} rows differ"
    assert np.array_equal(got2, want2), f"{case}, dim {dim}: second call on the same context differs"


def test_backward_with_skipped_lookups_at_the_borders():
    """Negative ids are skipped: their pairs sort behind every slot and form a run of their own, here one that
    begins inside a chunk, covers the next and ends in the third."""
    import paper_2204_05436_b200 as hl
    dim = 64
    ids, offsets, rows = _lookups([40, 8], seed=3)
    ids = np.concatenate([ids, np.full(70, -1, dtype=np.int32), np.full(9, 4, dtype=np.int32)])
    offsets = np.arange(len(ids) + 1, dtype=np.int32)
    rng = np.random.default_rng(9)
    cache = rng.integers(-8, 9, (rows, dim)).astype(np.float32)
    grad = rng.integers(-4, 5, (len(ids), dim)).astype(np.float32)
    want = cache.copy()
    keep = ids >= 0
    u, G = orc.row_gradients(ids[keep], np.arange(int(keep.sum()) + 1, dtype=np.int32), grad[keep])
    want[u] = (want[u].astype(np.float64) - 0.5 * G).astype(np.float32)
    got, _ = _backward(hl, ids, offsets, cache, grad, 0.5)
    assert np.array_equal(got, want)
