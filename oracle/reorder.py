"""CPU oracle of the reordering pre-pass (Data Reordering section): TEST INFRASTRUCTURE ONLY.

The paper sorts one dimension per iteration lexicographically by the coordinates of its entries in the
other dimensions, and all dimensions in turn, so that the entries gather around the diagonal. It gives no
more detail than that; the reading taken here keeps the FIRST element of each index's sorted entry list:

    one step for mode m:   key(x) = the smallest tuple (labels of the other modes, in increasing mode order)
                                    over the entries whose mode-m index is x; +infinity when x has no entry
                           the indices of mode m are re-numbered 0, 1, ... in ascending key order,
                           ties (and all empty indices) in the order of their current numbers
    one iteration:         a step for mode 0, then mode 1, ... each using the numbers the previous steps left
    result:                new_label[m][x] = the final number of original index x of mode m

Everything is integer work on plain numpy arrays, written step by step as above."""
from __future__ import annotations

import numpy as np


def reorder(coords, dims, iterations: int):
    order = len(dims)
    coords = [np.asarray(c, dtype=np.int64) for c in coords]
    n = len(coords[0]) if order else 0
    label = [np.arange(d, dtype=np.int64) for d in dims]            # current number of every original index
    for _ in range(iterations):
        for m in range(order):
            others = [o for o in range(order) if o != m]
            cur = label[m][coords[m]] if n else np.zeros(0, dtype=np.int64)       # current number of each entry's index
            # the tuple of the other modes' current numbers, as one integer (last mode varies fastest)
            tup = np.zeros(n, dtype=object)
            for o in others:
                tup = tup * int(dims[o]) + label[o][coords[o]].astype(object) if n else tup
            key = [None] * dims[m]                                                 # None = +infinity
            for e in range(n):
                x = int(cur[e])
                if key[x] is None or tup[e] < key[x]:
                    key[x] = tup[e]
            ranked = sorted(range(dims[m]), key=lambda x: (key[x] is None, key[x] if key[x] is not None else 0, x))
            renumber = np.empty(dims[m], dtype=np.int64)
            renumber[np.array(ranked, dtype=np.int64)] = np.arange(dims[m], dtype=np.int64)
            label[m] = renumber[label[m]]
    return [l.astype(np.int32) for l in label]


def window_columns(rows, cols, n_rows, window=64):
    """Locality measure used by the pins: the mean number of distinct columns touched by a window of
    consecutive rows (what a cache must hold while those rows are multiplied)."""
    rows, cols = np.asarray(rows), np.asarray(cols)
    total, count = 0, 0
    for s in range(0, n_rows, window):
        m = (rows >= s) & (rows < s + window)
        total += len(np.unique(cols[m]))
        count += 1
    return total / max(count, 1)
