"""Oracle of two further operations, in plain Python / numpy loops (TEST INFRASTRUCTURE ONLY, like the rest of
oracle/; shares nothing with the CUDA library):

  pack_ellpack   ELLPACK, which the paper's Tensor Storage Format section names among the formats that the four
                 level attributes compose. Reading used here (the paper does not spell the composition out): a
                 matrix with at most K entries per row is stored as THREE levels [D, D, S] -- the rows (dense),
                 K slots per row (dense; this level stores no tensor mode of its own), and one singleton
                 coordinate per slot, the entry's column. Row i's entries sit in its first slots, columns
                 ascending; unused slots hold column -1 and value 0. K is the longest row.
  elementwise    the element-wise product of the paper's Language section (`*` between operands whose indices
                 are not contraction indices): C_ij(k) = A_ij(k) * B_ij(k) with A sparse and B dense; the result
                 is sparse with A's structure.
"""
from __future__ import annotations

import numpy as np

from . import Packed, D, S


def pack_ellpack(coords, val, dims, mode_order=(0, 1)) -> Packed:
    rows_mode, cols_mode = mode_order
    M = int(dims[rows_mode])
    ri = np.asarray(coords[rows_mode], dtype=np.int64)
    ci = np.asarray(coords[cols_mode], dtype=np.int64)
    v = np.asarray(val, dtype=np.float64)
    per_row = [[] for _ in range(M)]
    for e in range(len(v)):                                  # every entry to its row, then each row by column
        per_row[ri[e]].append((int(ci[e]), float(v[e]), e))
    K = max((len(r) for r in per_row), default=0)
    crd = np.full(M * K, -1, dtype=np.int32)
    out = np.zeros(M * K, dtype=np.float64)
    perm = np.full(M * K, -1, dtype=np.int64)
    for i, r in enumerate(per_row):
        r.sort()
        for k, (c, x, e) in enumerate(r):
            if k > 0 and r[k - 1][0] == c:
                raise ValueError("duplicate coordinate")
            crd[i * K + k] = c
            out[i * K + k] = x
            perm[i * K + k] = e
    full_dims = (int(dims[0]), int(dims[1]), K)               # the slot level is described as a third "mode" of extent K
    empty = np.zeros(0, dtype=np.int32)
    return Packed(full_dims, (rows_mode, 2, cols_mode), (D, D, S),
                  [np.array([M], dtype=np.int32), np.array([K], dtype=np.int32), empty], [empty, empty, crd], out, perm)


def elementwise(coords, val, dims, B):
    """Per input entry e (in input order): val[e] * B[coords of e]; and the normaliser |val[e]| * |B[...]|."""
    B = np.asarray(B, dtype=np.float64)
    v = np.asarray(val, dtype=np.float64)
    out = np.zeros(len(v))
    norm = np.zeros(len(v))
    for e in range(len(v)):
        idx = tuple(int(np.asarray(c)[e]) for c in coords)
        out[e] = v[e] * B[idx]
        norm[e] = abs(v[e]) * abs(B[idx])
    return out, norm
