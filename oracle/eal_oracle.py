"""CPU oracle for the approximate access logger -- TEST INFRASTRUCTURE, not part of the product.

Only the tests, the smoke check and the benchmark's CPU-baseline leg may import this file.  It shares no code
with the CUDA library and never imports it.

What it models (Section V-B "Efficient Embedding Tracking", Section V-C for the randomizer): the Embedding Access
Logger is a cache-like structure of index tags with a 2-bit re-reference prediction value (RRPV) per block, replaced
by the Static Re-reference Interval Prediction policy (SRRIP), new blocks inserted one below the maximum RRPV; a
randomizer built as a Feistel network hashes the (index, table) tuple to spread the keys over the structure.  What
the logger holds at the end of the learning phase is the popular set.

The steps are taken one access at a time, in the order stated below, in plain Python.  The paper fixes the policy,
the counter width and the insertion value; the readings that are ours (associativity, victim order, hit promotion,
the order of accesses, the exact Feistel rounds) are stated where they are taken.

Pins (tests/test_eal_oracle.py): a hand-worked trace (tests/golden/srrip_trace.txt), the direct-mapped special case
(one way = the last key of each set), the FIFO behaviour of a pure scan, the no-eviction case (as many ways as distinct
keys), bijectivity of the randomizer, and the captured access mass against the exact counter on Zipf traffic.
Nothing in this file is "parity unpinned".
"""
from __future__ import annotations

from typing import Sequence

import numpy as np

RRPV_BITS = 2                        # Section V-B: "2-bit RRPV counter"
RRPV_MAX = (1 << RRPV_BITS) - 1      # 3: predicted re-reference in the distant future; also the value of empty ways
RRPV_INSERT = RRPV_MAX - 1           # 2: Section V-B, insertion one below the maximum ("long" interval in SRRIP)

_FEISTEL_KEYS = (0x85EBCA6B, 0xC2B2AE35, 0x27D4EB2F, 0x165667B1)
_FEISTEL_MUL = 0x9E3779B1


def randomizer(g) -> np.ndarray:
    """Section V-C: the randomizer hashes the (index, table) tuple -- here the global row g = base_t + index, which
    names the same tuple -- with a Feistel network.  Reading (the paper gives no rounds): four rounds on the 16-bit
    halves of the 32-bit key, round function F_r(x) = upper 16 bits of (x * 0x9E3779B1 + K_r) mod 2^32; a Feistel
    network is a bijection whatever F is."""
    g = np.asarray(g, dtype=np.uint64) & np.uint64(0xFFFFFFFF)
    left, right = g >> np.uint64(16), g & np.uint64(0xFFFF)
    for k in _FEISTEL_KEYS:
        f = ((right * np.uint64(_FEISTEL_MUL) + np.uint64(k)) & np.uint64(0xFFFFFFFF)) >> np.uint64(16)
        left, right = right, left ^ f
    return ((left << np.uint64(16)) | right).astype(np.uint32)


def set_of(g, n_sets: int) -> np.ndarray:
    """The set a key maps to: its randomized value modulo the number of sets."""
    return (randomizer(g).astype(np.int64) % int(n_sets)).astype(np.int64)


def tracker_new(n_sets: int, ways: int):
    """Empty logger: tags[set, way] = -1 (valid bit clear), rrpv = RRPV_MAX."""
    return (np.full((int(n_sets), int(ways)), -1, dtype=np.int64),
            np.full((int(n_sets), int(ways)), RRPV_MAX, dtype=np.int64))


def tracker_access(tags: np.ndarray, rrpv: np.ndarray, g: int) -> bool:
    """One access of key g under SRRIP with hit promotion; returns True on a hit.

    hit:   the block's RRPV becomes 0.
    miss:  the victim is the first way, from way 0 up, whose RRPV is RRPV_MAX (empty ways hold RRPV_MAX); while
           there is none every RRPV of the set is incremented; the victim takes tag g and RRPV_INSERT."""
    s = int(set_of(g, tags.shape[0]))
    ways = tags.shape[1]
    for w in range(ways):
        if tags[s, w] == g:
            rrpv[s, w] = 0
            return True
    while True:
        for w in range(ways):
            if rrpv[s, w] == RRPV_MAX:
                tags[s, w] = g
                rrpv[s, w] = RRPV_INSERT
                return False
        for w in range(ways):
            rrpv[s, w] += 1


def tracker_update(tags: np.ndarray, rrpv: np.ndarray, indices, offsets, batch: int, table_rows: Sequence[int],
                   bags_per_sample: int = 1) -> int:
    """The lookup engine hands the logger every index of every input (Section V-C).  Reading: the accesses of a
    mini-batch are taken in the order of its lookups in the table-major layout, j = 0 .. L-1 (the hardware's banked
    queue fixes no order); lookups whose index is outside its table are skipped.  Returns the number of hits."""
    indices = np.asarray(indices, dtype=np.int64)
    offsets = np.asarray(offsets, dtype=np.int64)
    rows = np.asarray(table_rows, dtype=np.int64)
    base = np.concatenate([[0], np.cumsum(rows)])
    T, B, S = len(rows), int(batch), int(bags_per_sample)
    hits = 0
    for bag in range(T * B * S):
        t = bag // (B * S)
        for j in range(int(offsets[bag]), int(offsets[bag + 1])):
            idx = int(indices[j])
            if idx < 0 or idx >= rows[t]:
                continue
            hits += bool(tracker_access(tags, rrpv, int(base[t]) + idx))
    return hits


def tracker_counts(tags: np.ndarray, rrpv: np.ndarray, total_rows: int) -> np.ndarray:
    """What the logger holds, as pseudo-counts for the popular-set selection: cnt[g] = RRPV_MAX + 1 - rrpv for every
    valid block (a block re-referenced recently weighs more), 0 for rows that are not tracked.  Selecting the popular
    rows from these counts with the rules of the exact counter keeps every tracked row if the capacity allows, and
    the most recently re-referenced ones otherwise."""
    cnt = np.zeros(int(total_rows), dtype=np.int64)
    valid = tags >= 0
    cnt[tags[valid]] = RRPV_MAX + 1 - rrpv[valid]
    return cnt


def captured_mass(hot_rows: np.ndarray, cnt_exact: np.ndarray) -> float:
    """Share of all counted accesses that go to the rows of a popular set (the measure behind the paper's comparison
    of the SRRIP logger with the exact one, Section V-B)."""
    total = float(np.sum(cnt_exact))
    return float(np.sum(cnt_exact[np.asarray(hot_rows, dtype=np.int64)])) / total if total else 0.0
