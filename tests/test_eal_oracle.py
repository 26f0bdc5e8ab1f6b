"""Pins of the access-logger oracle (oracle/eal_oracle.py) against facts that do not come from it."""
import os

import numpy as np

import gen
from oracle import eal_oracle as eal
from oracle import hotline_oracle as orc

HERE = os.path.dirname(os.path.abspath(__file__))


def test_hand_worked_trace_one_set_four_ways():
    tags, rrpv = eal.tracker_new(1, 4)
    with open(os.path.join(HERE, "golden", "srrip_trace.txt")) as f:
        lines = [ln.split() for ln in f if ln.strip() and not ln.startswith("#")]
    assert len(lines) == 15
    for step, (key, hit, *ways) in enumerate(lines):
        got_hit = eal.tracker_access(tags, rrpv, int(key))
        assert got_hit == bool(int(hit)), step
        for w, cell in enumerate(ways):
            tag, r = cell.split(":")
            assert tags[0, w] == (-1 if tag == "-" else int(tag)), (step, w)
            assert rrpv[0, w] == int(r), (step, w)


def test_one_way_is_a_direct_mapped_table_holding_the_last_key_of_each_set():
    rng = np.random.default_rng(5)
    keys = rng.integers(0, 5000, size=4000)
    n_sets = 97
    tags, rrpv = eal.tracker_new(n_sets, 1)
    for g in keys:
        eal.tracker_access(tags, rrpv, int(g))
    sets = eal.set_of(keys, n_sets)
    for s in range(n_sets):
        mine = keys[sets == s]
        assert tags[s, 0] == (mine[-1] if len(mine) else -1)


def test_a_scan_of_distinct_keys_replaces_ways_in_turn():
    # no key repeats: the policy degenerates to first-in first-out over the ways
    for ways in (1, 2, 4, 7):
        for n in (0, 1, ways - 1, ways, ways + 1, 3 * ways, 3 * ways + 2):
            if n < 0:
                continue
            tags, rrpv = eal.tracker_new(1, ways)
            for g in range(100, 100 + n):
                assert not eal.tracker_access(tags, rrpv, g)
            q, r = (n - 1) // ways, (n - 1) % ways + 1      # n = q*ways + r, 1 <= r <= ways (n >= 1)
            for w in range(ways):
                if n == 0:
                    assert tags[0, w] == -1 and rrpv[0, w] == 3
                elif w < r:
                    assert tags[0, w] == 100 + q * ways + w and rrpv[0, w] == 2
                elif q == 0:
                    assert tags[0, w] == -1 and rrpv[0, w] == 3
                else:
                    assert tags[0, w] == 100 + (q - 1) * ways + w and rrpv[0, w] == 3


def test_with_room_for_every_key_nothing_is_evicted():
    rng = np.random.default_rng(11)
    keys = rng.integers(0, 300, size=3000)
    n_sets = 8
    sets = eal.set_of(np.arange(300), n_sets)
    ways = int(np.bincount(sets, minlength=n_sets).max())
    tags, rrpv = eal.tracker_new(n_sets, ways)
    hits = sum(eal.tracker_access(tags, rrpv, int(g)) for g in keys)
    seen, times = np.unique(keys, return_counts=True)
    assert hits == len(keys) - len(seen)
    assert sorted(tags[tags >= 0].tolist()) == seen.tolist()
    for g, c in zip(seen, times):
        s = int(eal.set_of(g, n_sets))
        w = int(np.nonzero(tags[s] == g)[0][0])
        assert rrpv[s, w] == (0 if c >= 2 else 2)     # never aged: an empty way was always there


def _feistel_inverse(h):
    # undo the four rounds in reverse order with the same round function
    h = np.asarray(h, dtype=np.uint64)
    left, right = h >> np.uint64(16), h & np.uint64(0xFFFF)
    for k in (0x165667B1, 0x27D4EB2F, 0xC2B2AE35, 0x85EBCA6B):
        f = ((left * np.uint64(0x9E3779B1) + np.uint64(k)) & np.uint64(0xFFFFFFFF)) >> np.uint64(16)
        left, right = right ^ f, left
    return ((left << np.uint64(16)) | right).astype(np.uint32)


def test_randomizer_is_a_bijection_and_spreads_neighbouring_keys():
    g = np.concatenate([np.arange(1 << 20, dtype=np.uint32),
                        np.random.default_rng(2).integers(0, 1 << 32, size=1 << 18, dtype=np.uint64).astype(np.uint32)])
    h = eal.randomizer(g)
    assert len(np.unique(h)) == len(np.unique(g))
    assert np.array_equal(_feistel_inverse(h), g)
    # consecutive rows of one table land in all sets about equally often
    occ = np.bincount(eal.set_of(np.arange(1 << 16), 256), minlength=256)
    assert occ.min() > 0.7 * 256 and occ.max() < 1.3 * 256


def test_update_takes_the_lookups_in_layout_order_and_skips_bad_indices():
    spec = gen.CONFIGS["tiny"]
    geom = gen.make_geometry(spec)
    batch = gen.make_batch(spec, geom, 3)
    idx = batch.indices.copy()
    idx[5] = -1
    idx[9] = 10 ** 9
    g, _, _, t = orc.lookups_of(np.where((idx < 0) | (idx >= 10 ** 9), 0, idx), batch.offsets, spec.batch,
                                geom.table_rows, spec.bags_per_sample)
    ok = np.ones(len(idx), dtype=bool)
    ok[[5, 9]] = False
    a = eal.tracker_new(64, 4)
    b = eal.tracker_new(64, 4)
    hits_a = eal.tracker_update(a[0], a[1], idx, batch.offsets, spec.batch, geom.table_rows, spec.bags_per_sample)
    hits_b = sum(eal.tracker_access(b[0], b[1], int(x)) for x in g[ok])
    assert hits_a == hits_b
    assert np.array_equal(a[0], b[0]) and np.array_equal(a[1], b[1])


def test_logger_with_spare_capacity_captures_most_of_the_exact_popular_mass():
    # Zipf traffic: the rows the logger holds after the learning phase carry nearly the access mass of the same
    # number of exactly-counted top rows (Section V-B reports about 90 % of the exact logger on average)
    spec = gen.CONFIGS["tiny"]
    geom = gen.make_geometry(spec)
    batches = [gen.make_batch(spec, geom, i) for i in range(6)]
    cnt = orc.access_counts(((b.indices, b.offsets) for b in batches), spec.batch, geom.table_rows,
                            spec.bags_per_sample)
    N = int(sum(geom.table_rows))
    blocks = max(64, int(0.05 * N) // 16 * 16)
    tags, rrpv = eal.tracker_new(blocks // 16, 16)
    for b in batches:
        eal.tracker_update(tags, rrpv, b.indices, b.offsets, spec.batch, geom.table_rows, spec.bags_per_sample)
    marks = eal.tracker_counts(tags, rrpv, N)
    assert set(np.unique(marks)) <= {0, 1, 2, 3, 4}
    assert np.count_nonzero(marks) == np.count_nonzero(tags >= 0)
    k = int(0.7 * blocks)                                   # "70 % tracking capability"
    hot_tracked = orc.select_hot(marks, k)
    hot_exact = orc.select_hot(cnt, k)
    m_tracked, m_exact = eal.captured_mass(hot_tracked, cnt), eal.captured_mass(hot_exact, cnt)
    assert m_exact > 0.3
    assert m_tracked >= 0.85 * m_exact, (m_tracked, m_exact)
