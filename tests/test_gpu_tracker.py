"""The approximate access logger (hl_tracker_*) against its oracle: the tag and RRPV arrays must match bit for bit
after every mini-batch, whatever the shape of the logger, and the popular set selected from it must be the one the
oracle selects from its own logger."""
import dataclasses

import numpy as np
import pytest
import torch

import gen
from oracle import eal_oracle as eal
from oracle import hotline_oracle as orc
from harness import _t, max_nnz_of

pytestmark = pytest.mark.gpu


def _run(spec, n_sets, ways, n_batches=3, scale_rows=1.0, corrupt=False, select_k=()):
    import paper_2204_05436_b200 as hl
    geom = gen.make_geometry(spec, scale_rows)
    B, S, D = spec.batch, spec.bags_per_sample, spec.dim
    N = int(sum(geom.table_rows))
    max_nnz = max_nnz_of(spec, geom, B)
    host_table = torch.zeros((N, D), dtype=torch.float32).pin_memory()
    hot_cap = max(1, min(N, max(select_k) if select_k else 1))
    h = hl.Hotline(geom.table_rows, D, S, B, max_nnz, hot_cap, 1, host_table, device="cuda:0")
    tags_o, rrpv_o = eal.tracker_new(n_sets, ways)
    hits_o = 0
    try:
        with torch.cuda.stream(h.main):
            h.tracker_init(n_sets, ways)
            for i in range(n_batches):
                b = gen.make_batch(spec, geom, i)
                idx = b.indices.copy()
                if corrupt and len(idx) > 40:
                    idx[7] = -3
                    idx[33] = 2 ** 31 - 1
                hits_o += eal.tracker_update(tags_o, rrpv_o, idx, b.offsets, B, geom.table_rows, S)
                h.tracker_update(_t(idx.astype(np.int32), "cuda:0"), _t(b.offsets, "cuda:0"), B)
                h.synchronize()
                assert np.array_equal(h.trk_tags.cpu().numpy().reshape(n_sets, ways), tags_o), ("tags", i)
                assert np.array_equal(h.trk_rrpv.cpu().numpy().reshape(n_sets, ways), rrpv_o), ("rrpv", i)
                assert int(h.trk_hits.item()) == hits_o, ("hits", i)
            st = h.status(raise_on_error=False)
            assert st == (hl.HL_EBOUNDS if corrupt else hl.HL_OK)
            marks = eal.tracker_counts(tags_o, rrpv_o, N)
            for k in select_k:
                h.tracker_select(hl.HL_HOT_TOPK_ROWS, k)
                h.synchronize()
                n_hot = int(h.n_hot.item())
                want = orc.select_hot(marks, min(k, hot_cap))
                assert n_hot == len(want), ("n_hot", k)
                assert np.array_equal(h.hot_rows[:n_hot].cpu().numpy(), want), ("hot_rows", k)
        return dict(tracked=int(np.count_nonzero(tags_o >= 0)), hits=hits_o)
    finally:
        h.close()


@pytest.mark.parametrize("n_sets,ways", [(257, 4), (64, 16), (1, 32), (4096, 1), (1000, 7)])
def test_tracker_state_matches_the_oracle_access_by_access_order(n_sets, ways):
    stats = _run(gen.CONFIGS["tiny"], n_sets, ways)
    assert stats["hits"] > 0 and stats["tracked"] > 0


def test_tracker_with_bursts_of_one_row_and_repeats_inside_bags():
    # multi-hot bags of Zipf rows: long runs of one popular row inside a set, the case the replay skips through
    spec = dataclasses.replace(gen.CONFIGS["multi_hot"], batch=256, dim=16, rows=("fixed", 1500))
    stats = _run(spec, 16, 8, n_batches=2)
    assert stats["hits"] > stats["tracked"]


def test_tracker_skips_lookups_outside_their_table_and_reports_them():
    _run(gen.CONFIGS["tiny"], 128, 8, n_batches=2, corrupt=True)


def test_popular_set_selected_from_the_tracker():
    # fewer rows than tracked (the most recently re-referenced win, ties by row id), and more than tracked (all)
    _run(gen.CONFIGS["tiny"], 64, 16, n_batches=3, select_k=(100, 700, 5000))


def test_tracker_on_the_small_dlrm_shape():
    _run(gen.CONFIGS["dlrm_small"], 2048, 16, n_batches=2, scale_rows=0.02, select_k=(20000,))
