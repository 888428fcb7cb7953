"""Seeded index subsets for the random-k compressor (Def. 3).

The compressor keeps the entries of a k-element subset drawn uniformly from the k-subsets of a
segment.  The draw is an input of both implementations: this module samples it (numpy's
``Generator.choice`` without replacement, which is uniform over subsets) and sorts it; which
entries are then kept, and what happens to them, is not decided here.
"""
from __future__ import annotations

import numpy as np


def subset_seed(base_seed: int, row: int, step: int) -> int:
    """Distinct stream per (row, step); plain integer mixing."""
    return (int(base_seed) * 998_244_353 + int(step)) * 8191 + int(row) + 29


def random_subsets(seg_offsets, k, rows: int, step: int, base_seed: int) -> np.ndarray:
    """uint32 [rows, sum(k)]: for every row and segment t, k[t] distinct flat indices of that
    segment, ascending, drawn uniformly from its k[t]-subsets."""
    off = np.asarray(seg_offsets, dtype=np.int64)
    k = np.asarray(k, dtype=np.int64)
    assert off.size == k.size + 1 and off[-1] < 2 ** 32
    out = np.empty((rows, int(k.sum())), dtype=np.uint32)
    for r in range(rows):
        rng = np.random.default_rng(subset_seed(base_seed, r, step))
        q = 0
        for t in range(k.size):
            n, kt = int(off[t + 1] - off[t]), int(k[t])
            assert 1 <= kt <= n
            pick = np.sort(rng.choice(n, size=kt, replace=False, shuffle=False)) + off[t]
            out[r, q:q + kt] = pick.astype(np.uint32)
            q += kt
    return out
