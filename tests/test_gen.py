"""The synthetic-input generator: structure and distribution checks (CPU only)."""
import numpy as np
import pytest
import torch

import gen


@pytest.mark.parametrize("n_rows", [1, 2, 3, 5, 16, 17, 1000, 4099])
def test_feistel_is_a_bijection(n_rows):
    k = np.arange(n_rows)
    for key in (0, 1, 12345):
        img = gen.feistel_permute(k, n_rows, key)
        assert img.min() >= 0 and img.max() < n_rows
        assert np.array_equal(np.sort(img), k)
    if n_rows > 16:
        assert not np.array_equal(gen.feistel_permute(k, n_rows, 1), gen.feistel_permute(k, n_rows, 2))


def test_zipf_ranks_follow_the_bounded_law():
    rng = np.random.default_rng(7)
    R, alpha, n = 50, 1.1, 400_000
    ranks = gen.zipf_ranks(rng, alpha, R, n)
    assert ranks.min() >= 1 and ranks.max() <= R
    pmf = np.arange(1, R + 1, dtype=np.float64) ** -alpha
    pmf /= pmf.sum()
    freq = np.bincount(ranks, minlength=R + 1)[1:] / n
    sigma = np.sqrt(pmf * (1 - pmf) / n)
    assert (np.abs(freq - pmf) < 5 * sigma).all()
    uni = gen.zipf_ranks(rng, None, 10, 100_000)
    assert uni.min() == 1 and uni.max() == 10
    assert np.abs(np.bincount(uni)[1:] / 100_000 - 0.1).max() < 0.01


def test_table_values_numpy_and_torch_agree_and_are_on_the_grid():
    rows = np.arange(1000, 1300)
    for integer in (False, True):
        a = gen.table_values(rows, 16, seed=3, integer=integer)
        b = gen.table_values_torch(1000, 300, 16, 3, "cpu", integer=integer).numpy()
        assert a.dtype == np.float32 and np.array_equal(a, b)
    a = gen.table_values(rows, 16, 3)
    assert a.min() >= -0.5 and a.max() < 0.5
    assert np.array_equal(a * 2.0 ** 24, np.round(a * 2.0 ** 24))
    assert abs(float(a.mean())) < 0.02 and 0.07 < float(a.var()) < 0.095     # uniform: var 1/12
    big = gen.table_values(np.array([2 ** 31 + 5]), 64, 3)                    # counters beyond 32 bits
    assert np.array_equal(big, gen.table_values_torch(2 ** 31 + 5, 1, 64, 3, "cpu").numpy())
    ai = gen.table_values(rows, 16, 3, integer=True)
    assert ai.min() >= -512 and ai.max() <= 511 and np.array_equal(ai, np.round(ai))


@pytest.mark.parametrize("name", ["tiny", "tbsm"])
def test_batches_are_well_formed_and_reproducible(name):
    spec = gen.CONFIGS[name]
    geom = gen.make_geometry(spec)
    b0 = gen.make_batch(spec, geom, 0)
    b0_again = gen.make_batch(spec, geom, 0, threads=1)
    b1 = gen.make_batch(spec, geom, 1)
    assert np.array_equal(b0.indices, b0_again.indices) and np.array_equal(b0.offsets, b0_again.offsets)
    assert not np.array_equal(b0.indices, b1.indices)
    T, B, S = geom.num_tables, spec.batch, geom.bags_per_sample
    assert b0.offsets.shape[0] == T * B * S + 1 and b0.offsets[0] == 0 and b0.offsets[-1] == b0.nnz
    assert b0.indices.dtype == np.int32 and b0.offsets.dtype == np.int32
    per_table = b0.offsets[:: B * S]
    for t in range(T):
        seg = b0.indices[per_table[t]: per_table[t + 1]]
        assert seg.min() >= 0 and seg.max() < geom.table_rows[t]
    if name == "tbsm":   # one user per sample, repeated over the 21 steps
        users = b0.indices[: B * S].reshape(B, S)
        assert (users == users[:, :1]).all()


def test_multi_hot_bag_sizes():
    spec = gen.WorkloadSpec(name="mh", num_tables=2, dim=8, batch=4000, rows=("fixed", 1000), alpha=(1.05, 1.05),
                            pooling=("poisson", 20.0, 24), seed=5)
    geom = gen.make_geometry(spec)
    b = gen.make_batch(spec, geom, 0)
    sizes = np.diff(b.offsets)
    assert sizes.max() == 24 and sizes.min() >= 0
    assert 18.5 < sizes.mean() < 20.5        # Poisson(20) clipped at 24 loses a little mass


def test_geometry_of_the_named_configs():
    small = gen.make_geometry(gen.CONFIGS["dlrm_small"])
    large = gen.make_geometry(gen.CONFIGS["dlrm_large"])
    assert small.num_tables == 26 and abs(small.total_rows - 33.8e6) / 33.8e6 < 0.05
    assert large.num_tables == 26 and abs(large.total_rows - 266e6) / 266e6 < 0.05
    assert min(small.table_rows) >= 4 and max(small.table_rows) <= 10_000_000
    assert min(large.table_rows) >= 10 and max(large.table_rows) <= 40_000_000
    assert gen.make_geometry(gen.CONFIGS["tiny"]).base[-1] == 80_000
    avazu = gen.make_geometry(gen.CONFIGS["avazu_like"])
    assert avazu.num_tables == 21 and abs(avazu.total_rows - 9.3e6) / 9.3e6 < 0.01
    assert gen.CONFIGS["avazu_like"].n_dense == 1 and gen.CONFIGS["avazu_like"].dim == 16


def test_grad_values_streams():
    a = gen.grad_values(0, 0, 0, 100, 16)
    assert a.dtype == np.float32 and a.shape == (100, 16)
    assert not np.array_equal(a, gen.grad_values(0, 0, 1, 100, 16))
    gi = gen.grad_values(0, 0, 0, 100, 16, integer=True)
    assert np.array_equal(gi, np.round(gi)) and np.abs(gi).max() <= 8
