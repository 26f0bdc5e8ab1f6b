"""The named configurations at (or near) their full sizes: call by call and through Hotline.step (one mini-batch
after the other), and -- the DLRM-large-like one -- through the library's own scheduler, hl_pipe_*, which is the
launch configuration bench.py times."""
import dataclasses

import pytest

import gen
from tests.harness import run_config_check, run_fullsize_check, run_native_fullsize_check, run_pipelined_check

pytestmark = pytest.mark.gpu


def test_dlrm_large_full_size_sampled():
    """26 tables, 257.5 M rows x dim 64 (61 GiB pinned host table), batch 16,384: integer results in full,
    float results on samples."""
    stats = run_fullsize_check("dlrm_large")
    assert stats["N"] > 250_000_000 and 0 < stats["n_pop"] < stats["batch"] and stats["n_cold"] > 1000


def test_dlrm_large_full_size_through_the_benchmarked_schedule_bit_exact():
    """The same workload through NativePipelinedHotline (hl_pipe_*, index work two mini-batches ahead, order of
    Fig. 8) -- what bench.py times by default -- for five mini-batches on integer-valued tables and gradients:
    perm, counts, cold-row counts, every pooled vector, the whole hot cache and every written-back host row bit for
    bit against orc.hotline_step applied in sequence.  At this size the one-cluster cold-row search sees about
    18 K cold lookups, the movers choose their number of working CTAs, and both staging windows are in use."""
    stats = run_native_fullsize_check("dlrm_large", steps=5)
    assert stats["N"] > 250_000_000 and min(stats["n_cold"]) > 10_000
    assert all(0 < n < stats["batch"] for n in stats["n_pop"])


def test_tbsm_full_size_every_element():
    """3 tables (1 M, 4 M, 10 k rows), 21 time steps, batch 2,048, 64 MB budget: every output element."""
    stats = run_config_check("tbsm", steps=1)
    assert stats["N"] == 5_010_000


def test_dlrm_small_full_size_every_element():
    """26 tables, 33.8 M rows x dim 16, batch 4,096, 256 MB budget, 256 profiling batches: every output element."""
    stats = run_config_check("dlrm_small", steps=1)
    assert stats["N"] > 33_000_000 and stats["n_pop"] > 0


def test_avazu_like_full_size_every_element():
    """21 tables, 9.3 M rows x dim 16, one dense feature, batch 4,096, 128 MB budget: every output element, then
    three more mini-batches through the pipelined schedule."""
    stats = run_config_check("avazu_like", steps=1, profile_batches=32)
    assert abs(stats["N"] - 9.3e6) / 9.3e6 < 0.01 and stats["n_pop"] > 0
    run_pipelined_check("avazu_like", steps=3, integer=False, profile_batches=8)


def test_multi_hot_full_size_sampled():
    """8 tables x 20 M rows x dim 128 (76.3 GiB, one host allocation of 9.5 GiB per table), Poisson(20) bags capped
    at 64, the full batch of 65,536 inputs (10.5 M lookups): integer results in full, float results on samples."""
    stats = run_fullsize_check("multi_hot", n_samples=600, per_table=True)
    assert stats["batch"] == 65536 and stats["N"] == 160_000_000 and stats["n_cold"] > 1_000_000
