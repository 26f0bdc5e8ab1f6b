"""Pins of the CPU oracle to things other than itself (CPU only).

Each oracle function is checked against (a) a brute-force loop written here from the paper's definition,
(b) invariants and closed forms, (c) special cases that reduce to a library routine.  The paper prints no
worked numeric example for this path; tests/golden/ holds one small example worked by hand from the
definitions (see its header).
"""
import itertools
import os
from fractions import Fraction

import numpy as np
import pytest
import torch

import gen
from oracle import hotline_oracle as orc

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


# ----------------------------------------------------------------------------------------------------------
# tiny random mini-batches (independent of gen's Zipf machinery)
# ----------------------------------------------------------------------------------------------------------
def random_batch(rng, table_rows, B, S, max_pool, allow_empty=True):
    T = len(table_rows)
    sizes, idx = [], []
    for t in range(T):
        for _ in range(B * S):
            n = int(rng.integers(0 if allow_empty else 1, max_pool + 1))
            sizes.append(n)
            idx.extend(rng.integers(0, table_rows[t], n).tolist())
    offsets = np.concatenate([[0], np.cumsum(sizes)]).astype(np.int32)
    return np.asarray(idx, dtype=np.int32), offsets


def brute_lookups(indices, offsets, B, table_rows, S):
    """[(g, bag, sample, table)] by walking the CSR with plain loops."""
    base = [0]
    for r in table_rows:
        base.append(base[-1] + r)
    out = []
    for t in range(len(table_rows)):
        for b in range(B):
            for s in range(S):
                bag = (t * B + b) * S + s
                for j in range(offsets[bag], offsets[bag + 1]):
                    out.append((base[t] + int(indices[j]), bag, b, t))
    return out


CASES = [
    dict(table_rows=(5,), B=4, S=1, max_pool=1),
    dict(table_rows=(4, 3), B=6, S=1, max_pool=1),
    dict(table_rows=(6, 2, 7), B=8, S=1, max_pool=3),
    dict(table_rows=(5, 4), B=5, S=3, max_pool=2),
    dict(table_rows=(16, 9, 3), B=16, S=2, max_pool=4),
]


# ----------------------------------------------------------------------------------------------------------
# learning phase
# ----------------------------------------------------------------------------------------------------------
@pytest.mark.parametrize("case", CASES)
def test_access_counts_match_a_brute_force_tally(case):
    rng = np.random.default_rng(11)
    tr, B, S = case["table_rows"], case["B"], case["S"]
    batches = [random_batch(rng, tr, B, S, case["max_pool"]) for _ in range(3)]
    cnt = orc.access_counts(batches, B, tr, S)
    tally = [0] * sum(tr)
    for ind, off in batches:
        for g, _, _, _ in brute_lookups(ind, off, B, tr, S):
            tally[g] += 1
    assert cnt.tolist() == tally
    assert cnt.sum() == sum(len(i) for i, _ in batches)


def brute_select(cnt, k, share=None):
    total = sum(int(c) for c in cnt)
    cand = [g for g in range(len(cnt)) if cnt[g] >= 1]
    if share is not None:
        cand = [g for g in cand if Fraction(int(cnt[g]), total) >= Fraction(share[0], share[1])]
    cand.sort(key=lambda g: (-int(cnt[g]), g))
    return sorted(cand[:k])


def test_select_hot_ranking_ties_and_never_seen_rows():
    cnt = np.array([3, 0, 5, 3, 3, 0, 1, 5, 0, 3])
    assert orc.select_hot(cnt, 1).tolist() == [2]                 # 5 at rows 2 and 7: lower id wins
    assert orc.select_hot(cnt, 2).tolist() == [2, 7]
    assert orc.select_hot(cnt, 4).tolist() == [0, 2, 3, 7]        # ties at 3 broken by ascending id
    assert orc.select_hot(cnt, 100).tolist() == [0, 2, 3, 4, 6, 7, 9]   # rows with count 0 never enter
    assert orc.select_hot(cnt, 0).tolist() == []
    rng = np.random.default_rng(5)
    for _ in range(50):
        c = rng.integers(0, 4, rng.integers(1, 30))
        k = int(rng.integers(0, 35))
        assert orc.select_hot(c, k).tolist() == brute_select(c, k)
        hot = set(orc.select_hot(c, k).tolist())
        assert all(c[h] >= c[g] for h in hot for g in range(len(c)) if g not in hot and c[g] >= 1) or len(hot) == 0


def test_select_hot_min_share_is_exact_integer_arithmetic():
    # the paper's criterion: a popular row receives at least 1 of every 100,000 accesses
    cnt = np.zeros(50, dtype=np.int64)
    cnt[3], cnt[10], cnt[20], cnt[30] = 10, 9, 11, 999_970      # total = 1,000,000; 1e-5 share = 10 accesses
    assert orc.select_hot(cnt, 50, min_share=(1, 100_000)).tolist() == [3, 20, 30]
    assert orc.select_hot(cnt, 2, min_share=(1, 100_000)).tolist() == [20, 30]
    rng = np.random.default_rng(6)
    for _ in range(30):
        c = rng.integers(0, 50, 40)
        share = (int(rng.integers(1, 5)), int(rng.integers(20, 200)))
        assert orc.select_hot(c, 12, min_share=share).tolist() == brute_select(c, 12, share)


def test_hot_capacity_policies():
    assert orc.hot_capacity(("fraction", 5, 100), 80_000, 16) == 4_000
    assert orc.hot_capacity(("budget", 256 << 20), 10 ** 9, 16) == 4_194_304
    assert orc.hot_capacity(("budget", 1 << 30), 10 ** 9, 64) == 4_194_304
    assert orc.hot_capacity(("budget", 4 << 30), 10 ** 9, 128) == 8_388_608
    assert orc.hot_capacity(("budget", 1000), 10, 16) == 15       # floor(1000 / 64)
    assert orc.hot_capacity(("topk", 7), 10, 16) == 7


def test_remap_properties():
    hot = np.array([1, 4, 5, 9])
    remap = orc.build_remap(hot, 12)
    assert remap.dtype == np.int32 and remap.tolist() == [-1, 0, -1, -1, 1, 2, -1, -1, -1, 3, -1, -1]
    assert (remap[hot] == np.arange(4)).all() and (remap >= 0).sum() == 4
    table = np.arange(24, dtype=np.float32).reshape(12, 2)
    assert np.array_equal(orc.load_hot_cache(table, hot), table[[1, 4, 5, 9]])


# ----------------------------------------------------------------------------------------------------------
# fragment
# ----------------------------------------------------------------------------------------------------------
def brute_fragment(indices, offsets, B, table_rows, S, hot_set):
    """Loops only. Returns perm, n_pop, (O offsets, O ids as global rows), (X offsets, X ids as global rows)."""
    T = len(table_rows)
    base = [0]
    for r in table_rows:
        base.append(base[-1] + r)
    popular = []
    for b in range(B):
        ok = True
        for t in range(T):
            for s in range(S):
                bag = (t * B + b) * S + s
                for j in range(offsets[bag], offsets[bag + 1]):
                    if base[t] + int(indices[j]) not in hot_set:
                        ok = False
        popular.append(ok)
    O = [b for b in range(B) if popular[b]]
    X = [b for b in range(B) if not popular[b]]

    def emit(samples):
        off, ids = [0], []
        for t in range(T):
            for b in samples:
                for s in range(S):
                    bag = (t * B + b) * S + s
                    for j in range(offsets[bag], offsets[bag + 1]):
                        ids.append(base[t] + int(indices[j]))
                    off.append(len(ids))
        return off, ids

    return O + X, len(O), emit(O), emit(X)


def check_fragment(indices, offsets, B, tr, S, hot_rows):
    N = sum(tr)
    remap = orc.build_remap(np.asarray(sorted(hot_rows), dtype=np.int64), N)
    perm, n_pop, O, X, _ = orc.fragment(indices, offsets, B, tr, remap, S)
    bperm, bn, (boff, bids), (xoff, xids) = brute_fragment(indices, offsets, B, tr, S, set(hot_rows))
    assert perm.tolist() == bperm and n_pop == bn
    assert O.offsets.tolist() == boff and X.offsets.tolist() == xoff
    assert O.ids.tolist() == [int(remap[g]) for g in bids]         # popular: cache slots
    assert X.ids.tolist() == xids                                  # non-popular: global rows
    # Eq. 3: O and X partition M; order inside each is M's order
    assert sorted(perm.tolist()) == list(range(B))
    assert (np.diff(perm[:n_pop]) > 0).all() and (np.diff(perm[n_pop:]) > 0).all()
    assert (O.ids >= 0).all()
    return n_pop


@pytest.mark.parametrize("case", CASES)
def test_fragment_matches_brute_force_for_random_hot_sets(case):
    rng = np.random.default_rng(21)
    tr, B, S = case["table_rows"], case["B"], case["S"]
    N = sum(tr)
    for trial in range(20):
        ind, off = random_batch(rng, tr, B, S, case["max_pool"])
        frac = rng.random()
        hot = [g for g in range(N) if rng.random() < frac]
        check_fragment(ind, off, B, tr, S, hot)


def test_fragment_exhaustive_over_all_hot_sets():
    rng = np.random.default_rng(3)
    tr, B, S = (4, 3), 5, 1                       # N = 7 rows -> 128 hot sets
    ind, off = random_batch(rng, tr, B, S, 2)
    for mask in range(2 ** sum(tr)):
        hot = [g for g in range(sum(tr)) if mask >> g & 1]
        check_fragment(ind, off, B, tr, S, hot)


def test_fragment_degenerate_hot_sets():
    rng = np.random.default_rng(4)
    tr, B, S = (6, 5, 4), 12, 2
    ind, off = random_batch(rng, tr, B, S, 3, allow_empty=False)
    assert check_fragment(ind, off, B, tr, S, []) == 0                      # nothing hot: all inputs go to X
    assert check_fragment(ind, off, B, tr, S, list(range(sum(tr)))) == B    # all hot: all inputs popular
    # an input without any lookup is vacuously popular, even with an empty hot set
    off2 = off.copy()
    ind2, off2 = random_batch(rng, tr, B, S, 2, allow_empty=True)
    sizes = np.diff(off2).reshape(len(tr), B, S)
    empty_inputs = int((sizes.sum(axis=(0, 2)) == 0).sum())
    assert check_fragment(ind2, off2, B, tr, S, []) == empty_inputs


def test_fragment_and_cold_rows_keep_64_bit_row_ids_beyond_2_to_31():
    """Two tables with 2^31 + 90 rows together: the second table's rows have global ids that do not fit 32 bits.
    X's row ids, the cold rows and the unified slots against values worked out with Python integers."""
    tr = (2 ** 31 - 10, 100)
    N = sum(tr)
    B = 4
    # table 0: indices near both ends; table 1: every global id is >= 2^31 - 10
    ind = np.array([5, 2 ** 31 - 11, 7, 5, 0, 99, 50, 99], dtype=np.int32)
    off = np.arange(9, dtype=np.int32)
    hot = np.array([5, 2 ** 31 - 10 + 99], dtype=np.int64)          # one popular row per table
    remap = orc.build_remap(hot, N)
    perm, n_pop, O, X, _ = orc.fragment(ind, off, B, tr, remap, 1)
    # inputs: 0 -> rows (5, base+0), 1 -> (2^31-11, base+99), 2 -> (7, base+50), 3 -> (5, base+99): only input 3 is popular
    base1 = 2 ** 31 - 10
    assert perm.tolist() == [3, 0, 1, 2] and n_pop == 1
    assert O.ids.tolist() == [0, 1]
    assert X.ids.dtype == np.int64
    assert [int(v) for v in X.ids] == [5, 2 ** 31 - 11, 7, base1 + 0, base1 + 99, base1 + 50]
    C, slots = orc.gather_cold(X.ids, remap, 2)
    assert [int(v) for v in C] == [7, 2 ** 31 - 11, base1 + 0, base1 + 50]
    assert slots.tolist() == [0, 3, 2, 4, 1, 5]
    del remap


def test_fragment_dense_rows_follow_perm():
    rng = np.random.default_rng(8)
    tr, B = (5, 5), 9
    ind, off = random_batch(rng, tr, B, 1, 1, allow_empty=False)
    dense = rng.standard_normal((B, 3)).astype(np.float32)
    remap = orc.build_remap(np.array([0, 1, 2, 5, 6]), 10)
    perm, _, _, _, dense_out = orc.fragment(ind, off, B, tr, remap, 1, dense)
    for i in range(B):
        assert np.array_equal(dense_out[i], dense[perm[i]])


def test_all_hit_fraction_matches_the_zipf_closed_form():
    """Generator + fragment: with hot set = the top-h ranks of every table, an input is popular with
    probability prod_t (mass of ranks <= h in table t), independent lookups; the measured fraction must sit
    within 4 binomial sigma."""
    spec = gen.WorkloadSpec(name="cf", num_tables=4, dim=4, batch=20_000, rows=("list", (1000, 500, 2000, 50)),
                            alpha=(1.05, 1.2, 1.1, 1.3), seed=9)
    geom = gen.make_geometry(spec)
    batch = gen.make_batch(spec, geom, 0)
    top = (300, 200, 900, 20)
    hot, p_all = [], 1.0
    for t, (R, a, h) in enumerate(zip(geom.table_rows, spec.alpha, top)):
        pmf = np.arange(1, R + 1, dtype=np.float64) ** -a
        p_all *= pmf[:h].sum() / pmf.sum()
        key = int(np.random.default_rng([spec.seed, 0x7C9, t]).integers(0, 2 ** 31))
        hot.extend((geom.base[t] + gen.feistel_permute(np.arange(h), R, key)).tolist())
    remap = orc.build_remap(np.sort(np.asarray(hot)), geom.total_rows)
    _, n_pop, _, _, _ = orc.fragment(batch.indices, batch.offsets, spec.batch, geom.table_rows, remap)
    sigma = np.sqrt(p_all * (1 - p_all) / spec.batch)
    assert abs(n_pop / spec.batch - p_all) < 4 * sigma, (n_pop / spec.batch, p_all)


# ----------------------------------------------------------------------------------------------------------
# cold working set
# ----------------------------------------------------------------------------------------------------------
def test_gather_cold_properties_and_dereference():
    rng = np.random.default_rng(31)
    N, D, hot_cap = 60, 4, 20
    table = rng.standard_normal((N, D)).astype(np.float32)
    hot = np.sort(rng.choice(N, 15, replace=False))
    remap = orc.build_remap(hot, N)
    x_rows = rng.integers(0, N, 200)
    C, slots = orc.gather_cold(x_rows, remap, hot_cap)
    assert (np.diff(C) > 0).all()                                        # sorted, each cold row once
    assert set(C.tolist()) == set(x_rows.tolist()) - set(hot.tolist())   # disjoint from the hot set, complete
    assert C.tolist() == sorted(set(g for g in x_rows.tolist() if g not in set(hot.tolist())))
    cache = np.zeros((hot_cap + len(C), D), dtype=np.float32)
    cache[: len(hot)] = orc.load_hot_cache(table, hot)
    cache[hot_cap: hot_cap + len(C)] = orc.stage_cold_rows(table, C)
    assert np.array_equal(cache[slots], table[x_rows])                   # every lookup sees the table's bits
    for j, g in enumerate(x_rows.tolist()):
        assert slots[j] == (remap[g] if remap[g] >= 0 else hot_cap + C.tolist().index(g))
    # gather then scatter without an update leaves the table's bits alone
    t2 = table.copy()
    orc.scatter_cold(t2, C, cache[hot_cap:])
    assert np.array_equal(t2.view(np.uint32), table.view(np.uint32))
    # no cold rows at all
    C0, s0 = orc.gather_cold(hot[:5], remap, hot_cap)
    assert C0.shape == (0,) and s0.tolist() == list(range(5))


# ----------------------------------------------------------------------------------------------------------
# embedding bag forward / backward
# ----------------------------------------------------------------------------------------------------------
def brute_fwd(rows, ids, offsets):
    out = np.zeros((len(offsets) - 1, rows.shape[1]), dtype=np.float64)
    for bag in range(len(offsets) - 1):
        for j in range(offsets[bag], offsets[bag + 1]):
            for d in range(rows.shape[1]):
                out[bag, d] += float(rows[ids[j], d])
    return out


def random_csr(rng, n_bags, n_rows, max_pool):
    sizes = rng.integers(0, max_pool + 1, n_bags)
    offsets = np.concatenate([[0], np.cumsum(sizes)]).astype(np.int32)
    ids = rng.integers(0, n_rows, offsets[-1]).astype(np.int32)
    return ids, offsets


def test_embbag_fwd_matches_brute_force_and_torch():
    rng = np.random.default_rng(41)
    rows = rng.standard_normal((37, 8)).astype(np.float32)
    ids, offsets = random_csr(rng, 50, 37, 5)
    out = orc.embbag_fwd(rows, ids, offsets)
    assert out.dtype == np.float32
    assert np.array_equal(out, brute_fwd(rows, ids, offsets).astype(np.float32))
    ref = torch.nn.functional.embedding_bag(torch.from_numpy(ids.astype(np.int64)), torch.from_numpy(rows).double(),
                                            torch.from_numpy(offsets[:-1].astype(np.int64)), mode="sum").numpy()
    np.testing.assert_allclose(out, ref, rtol=1e-6, atol=1e-7)
    empty = np.flatnonzero(np.diff(offsets) == 0)
    assert len(empty) and (out[empty] == 0).all()


def test_embbag_fwd_pooling_one_is_a_row_gather_and_duplicates_count():
    rng = np.random.default_rng(42)
    rows = rng.standard_normal((20, 4)).astype(np.float32)
    ids = rng.integers(0, 20, 30).astype(np.int32)
    out = orc.embbag_fwd(rows, ids, np.arange(31, dtype=np.int32))
    assert np.array_equal(out.view(np.uint32), rows[ids].view(np.uint32))
    twice = orc.embbag_fwd(rows, np.array([3, 3, 3], dtype=np.int32), np.array([0, 3], dtype=np.int32))
    assert np.array_equal(twice[0], (3.0 * rows[3].astype(np.float64)).astype(np.float32))


def test_embbag_fwd_integer_tables_are_exact_in_any_order():
    rng = np.random.default_rng(43)
    rows = gen.table_values(np.arange(100), 8, 1, integer=True)
    ids, offsets = random_csr(rng, 40, 100, 64)
    out = orc.embbag_fwd(rows, ids, offsets)
    rev = np.zeros_like(out)
    for bag in range(40):
        for j in reversed(range(offsets[bag], offsets[bag + 1])):
            rev[bag] += rows[ids[j]]                       # fp32, reversed order: still exact
    assert np.array_equal(out, rev)


def brute_bwd(rows, ids, offsets, grad_out, lr):
    new = rows.astype(np.float64).copy()
    G = {}
    for bag in range(len(offsets) - 1):
        for j in range(offsets[bag], offsets[bag + 1]):
            G.setdefault(int(ids[j]), np.zeros(rows.shape[1]))
            G[int(ids[j])] = G[int(ids[j])] + grad_out[bag].astype(np.float64)
    lr64 = float(np.float32(lr))
    for u, g in G.items():
        new[u] = rows[u].astype(np.float64) - lr64 * g
    return new.astype(np.float32), G


def test_embbag_bwd_sgd_matches_brute_force_and_add_at():
    rng = np.random.default_rng(51)
    rows = rng.standard_normal((25, 6)).astype(np.float32)
    ids, offsets = random_csr(rng, 60, 25, 4)
    ids[:10] = 7                                           # a long duplicate run
    grad = rng.standard_normal((60, 6)).astype(np.float32)
    expect, G = brute_bwd(rows, ids, offsets, grad, 0.01)
    got = rows.copy()
    orc.embbag_bwd_sgd(got, ids, offsets, grad, 0.01)
    assert np.array_equal(got, expect)
    untouched = sorted(set(range(25)) - set(ids.tolist()))
    assert np.array_equal(got[untouched].view(np.uint32), rows[untouched].view(np.uint32))
    # library cross-check of the per-row gradient
    acc = np.zeros((25, 6))
    bag = np.repeat(np.arange(60), np.diff(offsets))
    np.add.at(acc, ids, grad[bag].astype(np.float64))
    u, Gm = orc.row_gradients(ids, offsets, grad)
    assert u.tolist() == sorted(G) and np.allclose(Gm, acc[u], rtol=1e-13, atol=1e-13)
    # conservation: sum of all row changes = lr * sum_bags |bag| * grad_out[bag]
    lhs = (rows.astype(np.float64) - got.astype(np.float64)).sum(axis=0)
    rhs = float(np.float32(0.01)) * (np.diff(offsets)[:, None] * grad.astype(np.float64)).sum(axis=0)
    np.testing.assert_allclose(lhs, rhs, atol=1e-5)


def test_embbag_bwd_sgd_special_cases():
    rng = np.random.default_rng(52)
    rows = rng.standard_normal((10, 4)).astype(np.float32)
    ids, offsets = random_csr(rng, 12, 10, 3)
    grad = rng.standard_normal((12, 4)).astype(np.float32)
    same = rows.copy()
    orc.embbag_bwd_sgd(same, ids, offsets, grad, 0.0)                     # lr = 0: bits unchanged
    assert np.array_equal(same.view(np.uint32), rows.view(np.uint32))
    # sign and scale: one lookup, lr = 0.5 -> row - 0.5 * grad
    one = rows.copy()
    orc.embbag_bwd_sgd(one, np.array([2], dtype=np.int32), np.array([0, 1], dtype=np.int32), grad[:1], 0.5)
    assert np.array_equal(one[2], (rows[2].astype(np.float64) - 0.5 * grad[0]).astype(np.float32))
    # integer data and lr = 2**-3: exact, any order
    irows = gen.table_values(np.arange(10), 4, 2, integer=True)
    igrad = gen.grad_values(0, 0, 0, 12, 4, integer=True)
    got = irows.copy()
    orc.embbag_bwd_sgd(got, ids, offsets, igrad, 0.125)
    exp = irows.copy()
    bag = np.repeat(np.arange(12), np.diff(offsets))
    for j in reversed(range(len(ids))):
        exp[ids[j]] -= np.float32(0.125) * igrad[bag[j]]                   # per-lookup fp32 updates: exact here
    assert np.array_equal(got, exp)
    # empty mini-batch
    orc.embbag_bwd_sgd(got, np.zeros(0, np.int32), np.zeros(1, np.int32), np.zeros((0, 4), np.float32), 0.1)


# ----------------------------------------------------------------------------------------------------------
# the pipeline invariant: fragmenting only rearranges inputs (Section I; Eq. 3-5)
# ----------------------------------------------------------------------------------------------------------
def run_both(rng, tr, B, S, D, max_pool, hot, integer):
    N = sum(tr)
    ind, off = random_batch(rng, tr, B, S, max_pool)
    table0 = gen.table_values(np.arange(N), D, 7, integer=integer)
    n_bags = len(tr) * B * S
    grad_full = gen.grad_values(1, 0, 2, n_bags, D, integer=integer)
    lr = 0.125 if integer else 0.01
    # baseline
    tb = table0.copy()
    pooled_b = orc.baseline_step(tb, ind, off, B, tr, S, grad_full, lr)
    # hotline, deferred order
    hot = np.asarray(sorted(hot), dtype=np.int64)
    remap = orc.build_remap(hot, N)
    hot_cap = len(hot) + 3
    cache = np.zeros((hot_cap + N, D), dtype=np.float32)
    cache[: len(hot)] = orc.load_hot_cache(table0, hot)
    perm, n_pop, O, X, _ = orc.fragment(ind, off, B, tr, remap, S)

    def mu_grad(samples):
        n = len(samples)
        src = ((np.arange(len(tr))[:, None, None] * B + np.asarray(samples, dtype=np.int64)[None, :, None]) * S
               + np.arange(S)[None, None, :]).reshape(-1)
        return grad_full[src], src

    g_pop, src_pop = mu_grad(perm[:n_pop])
    g_non, src_non = mu_grad(perm[n_pop:])
    th = table0.copy()
    out = orc.hotline_step(th, cache, hot_cap, remap, ind, off, B, tr, S, g_pop, g_non, lr, deferred=True)
    _, _, O2, X2, C, pooled_pop, pooled_non = out
    # un-permute pooled outputs
    pooled_h = np.zeros_like(pooled_b)
    pooled_h[src_pop] = pooled_pop
    pooled_h[src_non] = pooled_non
    # final table: host copy, with hot rows taken from the (authoritative) cache
    final = th.copy()
    final[hot] = cache[: len(hot)]
    assert set(C.tolist()).isdisjoint(set(hot.tolist()))
    return pooled_b, pooled_h, tb, final


@pytest.mark.parametrize("case", CASES)
@pytest.mark.parametrize("hot_kind", ["random", "empty", "full"])
def test_fragmented_step_equals_the_baseline_step(case, hot_kind):
    rng = np.random.default_rng(61)
    tr, B, S = case["table_rows"], case["B"], case["S"]
    N = sum(tr)
    hot = {"random": [g for g in range(N) if rng.random() < 0.6], "empty": [], "full": list(range(N))}[hot_kind]
    # integer data: bit-exact whatever the order of additions
    pb, ph, tb, th = run_both(rng, tr, B, S, 4, case["max_pool"], hot, integer=True)
    assert np.array_equal(pb, ph) and np.array_equal(tb, th)
    # real data: pooled outputs bit-equal (same per-bag order), tables within the fp32 tolerance
    pb, ph, tb, th = run_both(rng, tr, B, S, 4, case["max_pool"], hot, integer=False)
    assert np.array_equal(pb.view(np.uint32), ph.view(np.uint32))
    np.testing.assert_allclose(th, tb, rtol=1e-5, atol=1e-6)


# ----------------------------------------------------------------------------------------------------------
# hand-worked example (tests/golden/worked_example.txt)
# ----------------------------------------------------------------------------------------------------------
def _read_golden(path):
    vals = {}
    with open(path) as f:
        for line in f:
            line = line.split("#")[0].strip()
            if not line:
                continue
            key, rhs = line.split("=")
            vals[key.strip()] = [float(x) if "." in x else int(x) for x in rhs.split()]
    return vals


def test_hand_worked_example():
    g = _read_golden(os.path.join(GOLDEN, "worked_example.txt"))
    tr, B, S = tuple(g["table_rows"]), g["batch"][0], 1
    ind = np.asarray(g["indices"], dtype=np.int32)
    off = np.asarray(g["offsets"], dtype=np.int32)
    cnt = orc.access_counts([(ind, off)], B, tr, S)
    assert cnt.tolist() == g["counts"]
    hot = orc.select_hot(cnt, g["k"][0])
    assert hot.tolist() == g["hot_rows"]
    remap = orc.build_remap(hot, sum(tr))
    perm, n_pop, O, X, _ = orc.fragment(ind, off, B, tr, remap, S)
    assert perm.tolist() == g["perm"] and n_pop == g["n_pop"][0]
    assert O.offsets.tolist() == g["pop_offsets"] and O.ids.tolist() == g["pop_slots"]
    assert X.offsets.tolist() == g["non_offsets"] and X.ids.tolist() == g["non_rows"]
    C, slots = orc.gather_cold(X.ids, remap, g["hot_cap"][0])
    assert C.tolist() == g["cold_rows"] and slots.tolist() == g["non_slots"]
    table = np.asarray(g["table"], dtype=np.float32).reshape(sum(tr), 1)
    cache = np.zeros((g["hot_cap"][0] + len(C), 1), dtype=np.float32)
    cache[: len(hot)] = orc.load_hot_cache(table, hot)
    cache[g["hot_cap"][0]:] = orc.stage_cold_rows(table, C)
    assert orc.embbag_fwd(cache, O.ids, O.offsets)[:, 0].tolist() == g["pooled_pop"]
    assert orc.embbag_fwd(cache, slots, X.offsets)[:, 0].tolist() == g["pooled_non"]
    gp = np.asarray(g["grad_pop"], dtype=np.float32).reshape(-1, 1)
    gn = np.asarray(g["grad_non"], dtype=np.float32).reshape(-1, 1)
    orc.embbag_bwd_sgd(cache, O.ids, O.offsets, gp, g["lr"][0])
    orc.embbag_bwd_sgd(cache, slots, X.offsets, gn, g["lr"][0])
    assert cache[:, 0].tolist() == g["cache_after"]


def test_hand_worked_example_pins_the_order_of_a_step():
    """hotline_step as a whole, in both orders, against tests/golden/worked_example_order.txt: X looks up popular
    rows that O updates, so X's pooled vectors differ between the order of Fig. 8 (O forward, O update, X forward,
    X update: the default) and the order of Eq. 5 (both forwards first)."""
    g = _read_golden(os.path.join(GOLDEN, "worked_example_order.txt"))
    tr, B, S = tuple(g["table_rows"]), g["batch"][0], 1
    ind = np.asarray(g["indices"], dtype=np.int32)
    off = np.asarray(g["offsets"], dtype=np.int32)
    hot = np.asarray(g["hot_rows"], dtype=np.int64)
    hot_cap = g["hot_cap"][0]
    remap = orc.build_remap(hot, sum(tr))
    gp = np.asarray(g["grad_pop"], dtype=np.float32).reshape(-1, 1)
    gn = np.asarray(g["grad_non"], dtype=np.float32).reshape(-1, 1)
    assert g["pooled_non_fig8"] != g["pooled_non_eq5"]
    for deferred, key in ((False, "pooled_non_fig8"), (True, "pooled_non_eq5")):
        table = np.asarray(g["table"], dtype=np.float32).reshape(sum(tr), 1)
        cache = np.zeros((hot_cap + len(g["cold_rows"]), 1), dtype=np.float32)
        cache[: len(hot)] = orc.load_hot_cache(table, hot)
        perm, n_pop, O, X, C, pooled_pop, pooled_non = orc.hotline_step(
            table, cache, hot_cap, remap, ind, off, B, tr, S, gp, gn, g["lr"][0], deferred=deferred)
        assert perm.tolist() == g["perm"] and n_pop == g["n_pop"][0]
        assert O.offsets.tolist() == g["pop_offsets"] and O.ids.tolist() == g["pop_slots"]
        assert X.offsets.tolist() == g["non_offsets"] and X.ids.tolist() == g["non_slots"]
        assert C.tolist() == g["cold_rows"]
        assert pooled_pop[:, 0].tolist() == g["pooled_pop"]
        assert pooled_non[:, 0].tolist() == g[key], (deferred, pooled_non[:, 0].tolist())
        assert cache[:, 0].tolist() == g["cache_after"]
        assert table[:, 0].tolist() == g["table_after"]
    # the default is the order of Fig. 8
    table = np.asarray(g["table"], dtype=np.float32).reshape(sum(tr), 1)
    cache = np.zeros((hot_cap + len(g["cold_rows"]), 1), dtype=np.float32)
    cache[: len(hot)] = orc.load_hot_cache(table, hot)
    out = orc.hotline_step(table, cache, hot_cap, remap, ind, off, B, tr, S, gp, gn, g["lr"][0])
    assert out[6][:, 0].tolist() == g["pooled_non_fig8"]


def brute_step_fig8(table, indices, offsets, B, tr, S, hot_rows, grad_full, lr):
    """The step of Fig. 8 with plain loops over a dict of rows, no cache and no slots: O's bags are pooled, O's
    rows updated, then X's bags are pooled from the rows as they are now, then X's rows updated.  Returns pooled
    vectors in the mini-batch's own bag order and the final rows (fp64 arithmetic, rounded to fp32 per update)."""
    perm, n_pop, _, _ = brute_fragment(indices, offsets, B, tr, S, set(hot_rows))
    T, D = len(tr), table.shape[1]
    base = [0]
    for r in tr:
        base.append(base[-1] + r)
    rows = {g: table[g].astype(np.float32).copy() for g in range(sum(tr))}
    pooled = np.zeros((T * B * S, D), dtype=np.float32)
    lr64 = float(np.float32(lr))
    for samples in (perm[:n_pop], perm[n_pop:]):
        bags = [(t, (t * B + b) * S + s) for t in range(T) for b in samples for s in range(S)]
        for t, bag in bags:                                   # forward of this micro-batch
            acc = np.zeros(D, dtype=np.float64)
            for j in range(offsets[bag], offsets[bag + 1]):
                acc += rows[base[t] + int(indices[j])].astype(np.float64)
            pooled[bag] = acc.astype(np.float32)
        G = {}
        for t, bag in bags:                                   # its update: one per touched row
            for j in range(offsets[bag], offsets[bag + 1]):
                g = base[t] + int(indices[j])
                G[g] = G.get(g, np.zeros(D, dtype=np.float64)) + grad_full[bag].astype(np.float64)
        for g, grad in G.items():
            rows[g] = (rows[g].astype(np.float64) - lr64 * grad).astype(np.float32)
    return pooled, np.stack([rows[g] for g in range(sum(tr))])


@pytest.mark.parametrize("case", CASES)
def test_hotline_step_in_the_order_of_fig8_matches_a_brute_force_loop(case):
    """The default order (deferred=False) on random mini-batches and hot sets: pooled vectors and final rows equal
    a loop that runs O's forward and update before X's forward and update.  The hot sets are dense enough that X
    reads rows O has just updated, so the other order gives other pooled vectors (checked)."""
    rng = np.random.default_rng(67)
    tr, B, S = case["table_rows"], case["B"], case["S"]
    N, T, D = sum(tr), len(tr), 3
    differs = 0
    for trial in range(12):
        ind, off = random_batch(rng, tr, B, S, case["max_pool"])
        hot = np.asarray([g for g in range(N) if rng.random() < 0.75], dtype=np.int64)
        table0 = gen.table_values(np.arange(N), D, 13 + trial, integer=False)
        grad_full = gen.grad_values(5, trial, 2, T * B * S, D, integer=False)
        lr = 0.25
        want_pooled, want_rows = brute_step_fig8(table0, ind, off, B, tr, S, hot.tolist(), grad_full, lr)

        remap = orc.build_remap(hot, N)
        hot_cap = len(hot) + 2
        perm, n_pop, _, _, _ = orc.fragment(ind, off, B, tr, remap, S)

        def mu(samples):
            src = ((np.arange(T)[:, None, None] * B + np.asarray(samples, dtype=np.int64)[None, :, None]) * S
                   + np.arange(S)[None, None, :]).reshape(-1)
            return grad_full[src], src

        (g_pop, src_pop), (g_non, src_non) = mu(perm[:n_pop]), mu(perm[n_pop:])
        results = {}
        for deferred in (False, True):
            table = table0.copy()
            cache = np.zeros((hot_cap + N, D), dtype=np.float32)
            cache[: len(hot)] = orc.load_hot_cache(table0, hot)
            out = orc.hotline_step(table, cache, hot_cap, remap, ind, off, B, tr, S, g_pop, g_non, lr,
                                   deferred=deferred)
            pooled = np.zeros((T * B * S, D), dtype=np.float32)
            pooled[src_pop], pooled[src_non] = out[5], out[6]
            final = table.copy()
            final[hot] = cache[: len(hot)]
            results[deferred] = (pooled, final)
        assert np.array_equal(results[False][0].view(np.uint32), want_pooled.view(np.uint32)), trial
        assert np.array_equal(results[False][1].view(np.uint32), want_rows.view(np.uint32)), trial
        differs += not np.array_equal(results[True][0], want_pooled)
    # the two orders are told apart by these inputs (an input of X needs a popular and a non-popular lookup for that)
    assert differs > 0 or T * S * case["max_pool"] == 1


def test_input_record_size_matches_the_papers_buffer_sizing():
    """Section V-A: a 2.5 MB input buffer holds mini-batches of up to 16 K inputs, i.e. 160 bytes per input;
    26 four-byte sparse indices + 13 four-byte dense features + a four-byte label is exactly that, which is
    why the boundary takes int32 indices and fp32 dense features."""
    per_input = int(2.5 * 2 ** 20) // (16 * 1024)
    assert per_input == 160 == 26 * 4 + 13 * 4 + 4
    assert gen.make_batch(gen.CONFIGS["tiny"], gen.make_geometry(gen.CONFIGS["tiny"]), 0).indices.itemsize == 4


def test_flush_hot_gives_a_consistent_table():
    rng = np.random.default_rng(71)
    table = rng.standard_normal((30, 3)).astype(np.float32)
    hot = np.array([2, 5, 11, 29])
    cache = np.zeros((6, 3), dtype=np.float32)
    cache[:4] = orc.load_hot_cache(table, hot) + 1.0          # the cache moved on; the host copies are stale
    cache[4:] = 99.0                                          # unused slots and staging must not leak
    before = table.copy()
    orc.flush_hot(table, cache, hot)
    assert np.array_equal(table[hot], before[hot] + 1.0)
    rest = np.setdiff1d(np.arange(30), hot)
    assert np.array_equal(table[rest].view(np.uint32), before[rest].view(np.uint32))
