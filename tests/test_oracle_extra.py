"""Pins of the ELLPACK packing and of the element-wise product of the oracle (CPU only)."""
import numpy as np
import pytest
import scipy.sparse as sp

import oracle
import synth
from oracle import D, CU, S
from oracle import extra
from table1 import enumerate_entries


def _np(coords):
    return [c.numpy() for c in coords]


def test_ellpack_worked_example():
    """The 4 x 6 matrix of the other worked examples: rows of 2, 0, 3 and 1 entries, so K = 3."""
    c = ([0, 0, 2, 2, 2, 3], [4, 1, 5, 0, 1, 3])
    v = [2.0, 1.0, 5.0, 3.0, 4.0, 6.0]
    pk = extra.pack_ellpack(c, v, (4, 6))
    assert pk.attr == (D, D, S) and pk.mode_order == (0, 2, 1) and pk.dims == (4, 6, 3)
    assert pk.pos[0].tolist() == [4] and pk.pos[1].tolist() == [3]
    assert pk.crd[2].tolist() == [1, 4, -1, -1, -1, -1, 0, 1, 5, 3, -1, -1]
    assert pk.val.tolist() == [1, 2, 0, 0, 0, 0, 3, 4, 5, 6, 0, 0]


@pytest.mark.parametrize("dims,nnz,seed", [((64, 48), 700, 1), ((300, 200), 900, 2), ((1, 500), 300, 3), ((500, 1), 200, 4),
                                           ((40, 40), 1600, 5), ((20, 30), 0, 6)])
def test_ellpack_against_the_level_reader_and_scipy(dims, nnz, seed):
    coords, val = synth.random_coo(dims, nnz, seed)
    c, v = _np(coords), val.numpy()
    pk = extra.pack_ellpack(c, v, dims)
    M, K = dims[0], pk.dims[2]
    assert K == (np.bincount(c[0], minlength=M).max() if nnz else 0)
    # the level rules of the storage format, walked by the independent reader: every (row, slot) position once
    walked = enumerate_entries(pk.attr, pk.pos, pk.crd)
    assert [p for p, _ in walked] == list(range(M * K))
    stored = [(i, col) for _, (i, _, col) in walked if col >= 0]
    assert sorted(stored) == sorted(zip(c[0].tolist(), c[1].tolist())) and len(set(stored)) == len(stored)
    for p, (i, k, col) in walked:
        assert p == i * K + k
        if col < 0:
            assert pk.val[p] == 0.0 and all(pk.crd[2][q] < 0 for q in range(p, (i + 1) * K))      # padding only at the end
        elif k > 0:
            assert pk.crd[2][p - 1] < col                                                          # ascending inside a row
    # the matrix it stores is the input matrix
    keep = pk.crd[2] >= 0
    rows = np.repeat(np.arange(M), K)[keep]
    got = sp.coo_matrix((pk.val[keep], (rows, pk.crd[2][keep])), shape=dims).toarray()
    want = sp.coo_matrix((v, (c[0], c[1])), shape=dims).toarray()
    assert np.array_equal(got, want)
    # same slots as the CSR packing, row by row
    csr = oracle.pack(c, v, dims, (0, 1), (D, CU))
    for i in range(M):
        a, b = csr.pos[1][i], csr.pos[1][i + 1]
        assert pk.crd[2][i * K:i * K + (b - a)].tolist() == csr.crd[1][a:b].tolist()
    # input order does not matter
    perm = np.random.default_rng(seed).permutation(len(v))
    pk2 = extra.pack_ellpack([x[perm] for x in c], v[perm], dims)
    assert np.array_equal(pk2.crd[2], pk.crd[2]) and np.array_equal(pk2.val, pk.val)


@pytest.mark.parametrize("dims", [(7, 6), (5, 4, 3), (3, 4, 2, 5)])
def test_elementwise_against_dense(dims):
    nnz = int(np.prod(dims)) // 2
    coords, val = synth.random_coo(dims, nnz, 9)
    c, v = _np(coords), val.numpy()
    B = synth.random_dense(dims, 9).numpy()
    got, norm = extra.elementwise(c, v, dims, B)
    dense = np.zeros(dims)
    dense[tuple(c)] = v
    want = (dense * B)[tuple(c)]                              # numpy's own element-wise product, read back at the entries
    assert np.array_equal(got, want)
    assert np.array_equal(norm, np.abs(want))
    ones, _ = extra.elementwise(c, v, dims, np.ones(dims))    # B = 1 returns A's values
    assert np.array_equal(ones, v)
    assert not extra.elementwise(c, v, dims, np.zeros(dims))[0].any()
