"""CUDA path vs CPU oracle, call by call, through the C boundary (needs a B200)."""
import dataclasses

import numpy as np
import pytest
import torch

import gen
from tests.harness import run_config_check, run_pipelined_check, run_recalibration_check

pytestmark = pytest.mark.gpu


def test_tiny_config():
    stats = run_config_check("tiny", steps=3)
    assert 0 < stats["n_pop"] < stats["batch"]


def test_tiny_config_three_steps_without_resync():
    """The two sides are never re-aligned: their rounding differences accumulate over the steps and must still
    stay inside the tolerance on this pooling-1 workload."""
    run_config_check("tiny", steps=3, resync=False)


def test_tiny_config_deferred_order_and_no_overlap():
    run_config_check("tiny", steps=2, deferred=True, overlap=False)


def test_tiny_integer_data_is_bit_exact():
    run_config_check("tiny", steps=2, integer=True)


@pytest.mark.parametrize("hot", ["empty", "full", ("random", 0.3), ("random", 0.9)])
def test_arbitrary_hot_sets(hot):
    """Misclassifying a row never changes the result (Section V-B): any hot set must give the oracle's answer."""
    spec = dataclasses.replace(gen.CONFIGS["tiny"], hot_policy=("topk", 80_000))
    stats = run_config_check(spec, steps=2, hot_override=hot)
    if hot == "empty":
        assert stats["n_pop"] == 0
    if hot == "full":
        assert stats["n_non"] == 0 and stats["n_cold"] == 0


@pytest.mark.parametrize("batch", [2559, 2560, 2561, 3000, 5119, 5120, 5121, 6000])
def test_cold_row_search_at_the_limit_of_its_one_cluster_path(batch):
    """Empty hot set, 8 tables: every lookup is cold, 8 * batch of them.  The one-cluster kernel takes at most 40 960
    (a cluster of 16 CTAs; 20 480 where the device places only 8); one more and the general path (tile sort, head
    flags, scan, assignment), launched from the device, does the work."""
    spec = dataclasses.replace(gen.CONFIGS["tiny"], batch=batch, hot_policy=("topk", 80_000))
    stats = run_config_check(spec, steps=2, hot_override="empty", integer=True)
    assert stats["n_pop"] == 0 and stats["n_cold"] > 5_000        # distinct rows; the lookups are 8 * batch


def test_one_host_allocation_per_table():
    """hl_set_host_tables: every table in an allocation of its own (ragged sizes), the call-by-call path and the
    library's scheduler both bit-exact on integer data."""
    spec = gen.WorkloadSpec(name="ragged_tables", num_tables=11, dim=32, batch=777, rows=("loguniform", 4, 30_000, 3),
                            alpha=tuple([1.1] * 11), hot_policy=("fraction", 10, 100), profile_batches=4, seed=23)
    run_config_check(spec, steps=2, integer=True, per_table=True)
    run_config_check(spec, steps=1, per_table=True)
    run_pipelined_check(spec, steps=5, integer=True, native=True, per_table=True)


def test_min_share_policy():
    spec = dataclasses.replace(gen.CONFIGS["tiny"], hot_policy=("share", 1, 2000))
    run_config_check(spec, steps=1)


@pytest.mark.parametrize("dim", [4, 8, 32, 64, 128, 200])
def test_row_widths(dim):
    spec = dataclasses.replace(gen.CONFIGS["tiny"], dim=dim, batch=333, rows=("fixed", 3001))
    run_config_check(spec, steps=2)


def test_ragged_shapes_many_tables():
    spec = gen.WorkloadSpec(name="ragged", num_tables=37, dim=16, batch=1237, rows=("loguniform", 4, 50_000, 7),
                            alpha=tuple([1.1] * 37), n_dense=5, hot_policy=("fraction", 20, 100), profile_batches=6,
                            seed=11)
    run_config_check(spec, steps=2)


def test_multi_hot_bags():
    spec = dataclasses.replace(gen.CONFIGS["multi_hot"], batch=2048, rows=("fixed", 50_000),
                               hot_policy=("fraction", 30, 100), profile_batches=4)
    stats = run_config_check(spec, steps=2)
    assert stats["L_non"] > 0


def test_multi_hot_integer_data_long_runs():
    spec = dataclasses.replace(gen.CONFIGS["multi_hot"], batch=4096, dim=64, rows=("fixed", 500),
                               hot_policy=("fraction", 50, 100), profile_batches=2)
    run_config_check(spec, steps=1, integer=True)


def test_time_series_shape():
    spec = dataclasses.replace(gen.CONFIGS["tbsm"], batch=512, rows=("list", (20_000, 80_000, 1000)),
                               hot_policy=("fraction", 60, 100), profile_batches=8)
    stats = run_config_check(spec, steps=2)
    assert stats["n_pop"] > 0


def test_dlrm_small_scaled():
    stats = run_config_check("dlrm_small", steps=2, scale_rows=0.05, profile_batches=8)
    assert stats["n_pop"] > 0 and stats["n_cold"] > 0


def test_dlrm_large_scaled():
    spec = dataclasses.replace(gen.CONFIGS["dlrm_large"], batch=4096)
    run_config_check(spec, steps=1, scale_rows=0.002, profile_batches=4)


def test_batch_of_one_and_single_table():
    spec = gen.WorkloadSpec(name="one", num_tables=1, dim=16, batch=1, rows=("fixed", 50), alpha=(1.5,),
                            hot_policy=("topk", 10), profile_batches=3, seed=3)
    run_config_check(spec, steps=2)


def test_pipelined_steps_equal_sequential_steps_integer_data():
    """Six mini-batches through the software pipeline; with integer data the result must be bit-identical to the
    oracle's one-after-the-other processing.  Consecutive Zipf mini-batches share cold rows, so this exercises the
    forwarding of staged rows and the ordering of write-backs."""
    stats = run_pipelined_check("tiny", steps=6, integer=True)
    assert stats["shared_cold_rows"] > 50


def test_pipelined_steps_without_sorting_ahead_integer_data():
    """The pipeline with the backward sorts left on the main stream (hl_embbag_bwd_sgd instead of prepare/apply)."""
    stats = run_pipelined_check("tiny", steps=6, integer=True, sort_ahead=False)
    assert stats["shared_cold_rows"] > 50


def test_pipelined_steps_with_index_work_one_mini_batch_ahead_integer_data():
    """lookahead=1: fragment, cold-row search and sort of mini-batch j+1 are issued during mini-batch j (the default
    issues them during j-1)."""
    stats = run_pipelined_check("tiny", steps=6, integer=True, lookahead=1)
    assert stats["shared_cold_rows"] > 50
    run_pipelined_check("dlrm_small", steps=3, scale_rows=0.02, integer=False, profile_batches=6, lookahead=1)


def test_pipelined_steps_with_one_sort_per_micro_batch_integer_data():
    """Sorting ahead with hl_embbag_bwd_prepare / apply per micro-batch instead of the combined sort of O and X."""
    stats = run_pipelined_check("tiny", steps=6, integer=True, combined_sort=False)
    assert stats["shared_cold_rows"] > 50
    spec = dataclasses.replace(gen.CONFIGS["multi_hot"], batch=512, dim=32, rows=("fixed", 2000),
                               hot_policy=("fraction", 40, 100), profile_batches=2)
    run_pipelined_check(spec, steps=4, integer=True, combined_sort=False)


def test_pipelined_steps_with_serialised_link_integer_data():
    """The default schedule of the pipeline: the next mini-batch's host rows are read after this one's write-back."""
    run_pipelined_check("tiny", steps=6, integer=True, overlap_link=False)
    spec = dataclasses.replace(gen.CONFIGS["multi_hot"], batch=512, dim=32, rows=("fixed", 2000),
                               hot_policy=("fraction", 40, 100), profile_batches=2)
    run_pipelined_check(spec, steps=4, integer=True, overlap_link=False)


def test_pipelined_steps_real_data_and_dense_features():
    run_pipelined_check("dlrm_small", steps=3, scale_rows=0.02, integer=False, profile_batches=6)


def test_pipelined_multi_hot_integer_data():
    spec = dataclasses.replace(gen.CONFIGS["multi_hot"], batch=1024, dim=32, rows=("fixed", 3000),
                               hot_policy=("fraction", 40, 100), profile_batches=2)
    stats = run_pipelined_check(spec, steps=5, integer=True)
    assert stats["shared_cold_rows"] > 100


def test_native_pipeline_equals_sequential_steps_integer_data():
    """The same schedule issued by the library itself (hl_pipe_*): bit-identical to the oracle's one-after-the-other
    processing on integer data, with forwarding of shared cold rows, for index work one, two and three mini-batches
    ahead."""
    for ahead in (1, 2, 3):
        stats = run_pipelined_check("tiny", steps=7, integer=True, native=True, lookahead=ahead)
        assert stats["shared_cold_rows"] > 50
    spec = dataclasses.replace(gen.CONFIGS["multi_hot"], batch=512, dim=32, rows=("fixed", 2000),
                               hot_policy=("fraction", 40, 100), profile_batches=2)
    run_pipelined_check(spec, steps=4, integer=True, native=True)


def test_native_pipeline_queues_the_same_launches_whichever_cold_row_search_runs():
    """The host queues the same kernels for every mini-batch: when a mini-batch has more cold lookups than the
    one-cluster kernel takes, that kernel launches the general search (tile sort, head flags, scan, assignment) from
    the device.  Same results either way, and the host-side launch count does not depend on the data or on whether the
    host waits between steps."""
    kw = dict(steps=6, scale_rows=0.02, integer=True, profile_batches=6, native=True)
    few = run_pipelined_check("dlrm_small", drain_between=True, **kw)      # a few thousand cold lookups per mini-batch
    spec = dataclasses.replace(gen.CONFIGS["multi_hot"], batch=2048, dim=32, rows=("fixed", 20000),
                               hot_policy=("fraction", 10, 100), profile_batches=2)
    a = run_pipelined_check(spec, steps=4, integer=True, native=True)      # tens of thousands: the general search
    b = run_pipelined_check(spec, steps=4, integer=True, native=True, drain_between=True)
    assert a["launches"] == b["launches"] and few["launches"] > 0


@pytest.mark.parametrize("native", [False, True])
def test_pipelines_with_an_empty_micro_batch(native):
    """No popular row at all (O is empty, every lookup is cold), and tables so small that the learning phase sees
    every row (X is empty, nothing crosses the host link): both schedulers, bit-exact on integer data."""
    none_hot = dataclasses.replace(gen.CONFIGS["tiny"], batch=256, hot_policy=("topk", 0), profile_batches=2)
    stats = run_pipelined_check(none_hot, steps=4, integer=True, native=native)
    assert stats["shared_cold_rows"] > 0
    all_hot = dataclasses.replace(gen.CONFIGS["tiny"], batch=256, rows=("fixed", 40), hot_policy=("fraction", 100, 100),
                                  profile_batches=8)
    stats = run_pipelined_check(all_hot, steps=4, integer=True, native=native)
    assert stats["shared_cold_rows"] == 0


@pytest.mark.parametrize("write_back", ["exclusive", "after_forward"])
def test_native_pipeline_write_back_modes(write_back):
    """hl_pipe_options.write_back: the write-back of a mini-batch alone on the chip, or held over until the next
    mini-batch's popular forward is over (queued by the next step, by a drain between steps, or at once by the last
    step): the same results, bit for bit on integer data, with rows forwarded between consecutive mini-batches."""
    assert run_pipelined_check("tiny", steps=7, integer=True, native=True, write_back=write_back)["shared_cold_rows"] > 50
    run_pipelined_check("tiny", steps=5, integer=True, native=True, write_back=write_back, drain_between=True)
    run_pipelined_check("tiny", steps=5, integer=True, native=True, write_back=write_back, lookahead=1)
    run_pipelined_check("dlrm_small", steps=4, scale_rows=0.02, integer=True, profile_batches=6, native=True,
                        write_back=write_back, lookahead=3)
    if write_back == "after_forward":
        run_pipelined_check("tiny", steps=6, integer=True, native=True, write_back=write_back, order="eq5")


def test_native_pipeline_in_the_order_of_eq5_one_update_per_row_and_mini_batch():
    """Both forwards, then one update of every touched row with the gradient of the whole mini-batch (the lookups of a
    row from O and from X form one run of the merged sort): bit-exact on integer data, within the tolerance on real
    data, with rows that O and X share (hot rows) and rows that consecutive mini-batches share (forwarded)."""
    assert run_pipelined_check("tiny", steps=6, integer=True, native=True, order="eq5")["shared_cold_rows"] > 50
    spec = dataclasses.replace(gen.CONFIGS["multi_hot"], batch=512, dim=32, rows=("fixed", 2000),
                               hot_policy=("fraction", 40, 100), profile_batches=2)
    run_pipelined_check(spec, steps=4, integer=True, native=True, order="eq5")
    run_pipelined_check("dlrm_small", steps=3, scale_rows=0.02, integer=False, profile_batches=6, native=True,
                        order="eq5")


def test_native_pipeline_refuses_what_it_cannot_queue():
    """hl_pipe_step before any hl_pipe_submit, and more submissions than there are spare buffer sets."""
    import numpy as np
    import torch
    import paper_2204_05436_b200 as hl
    spec = gen.CONFIGS["tiny"]
    geom = gen.make_geometry(spec)
    B, D = spec.batch, spec.dim
    N = int(sum(geom.table_rows))
    n_bags = geom.num_tables * B
    table = torch.zeros((N, D), dtype=torch.float32).pin_memory()
    p = hl.NativePipelinedHotline(geom.table_rows, D, 1, B, n_bags, 4096, 4096, table, lookahead=2)
    try:
        with torch.cuda.stream(p.main):
            p.set_hot_rows(torch.arange(100, dtype=torch.int32, device="cuda:0"))
            p.build_remap(load_rows=True)
            b = gen.make_batch(spec, geom, 0)
            idx = torch.from_numpy(b.indices).to("cuda:0")
            off = torch.from_numpy(b.offsets).to("cuda:0")
            grad = torch.zeros((n_bags, D), device="cuda:0")
            with pytest.raises(hl.HotlineError):
                p.step(grad, grad, 0.1)                       # nothing submitted
            p.start(idx, off, B, None, more=[(idx, off, B, None), (idx, off, B, None)])   # 3 of 4 sets
            with pytest.raises(hl.HotlineError):
                hl.hl_pipe_submit(p.pipe, p._batch(idx, off, B), None)                   # no spare set left
            for _ in range(3):
                p.step(grad, grad, 0.1)
            p.drain()
            assert p.status() == hl.HL_OK
    finally:
        p.close()


def test_native_pipeline_real_data_and_dense_features():
    run_pipelined_check("dlrm_small", steps=3, scale_rows=0.02, integer=False, profile_batches=6, native=True)


def test_flush_and_second_learning_phase():
    """Re-calibration: flush the popular rows, learn another popular set from later mini-batches, carry on."""
    stats = run_recalibration_check("tiny")
    assert stats["hot_sets_differ"]
