"""Pins for the oracle's format packing: Table 1's loops (an independent reader), scipy's COO->CSR
conversion, structural invariants, a hand-worked example, shuffle invariance and rejected inputs."""
import numpy as np
import pytest
import scipy.sparse as sp

import oracle
import synth
from oracle import D, CU, CN, S
from table1 import enumerate_entries

FORMATS_2D = {"COO": (CN, S), "CSR": (D, CU), "DCSR": (CU, CU)}
FORMATS_3D = {"COO": (CN, S, S), "CSF": (CU, CU, CU), "DCSF": (D, CU, CU)}


def _np(coords):
    return [c.numpy() for c in coords]


def _sorted_entries(coords, val, mode_order):
    """The input entries, sorted lexicographically in storage order: (coords in level order, value)."""
    cols = [np.asarray(coords[m]) for m in mode_order]
    perm = np.lexsort(cols[::-1])
    return [tuple(int(c[p]) for c in cols) for p in perm], np.asarray(val)[perm]


# --- hand-worked example. Derived by hand from the attribute definitions and Table 1's loop forms
# (the paper's own example figure is not reproduced in its text): a 4x6 matrix with row 1 empty.
M_COORDS = ([0, 0, 2, 2, 2, 3], [1, 4, 0, 1, 5, 3])
M_VAL = [1.0, 2.0, 3.0, 4.0, 5.0, 6.0]
M_DIMS = (4, 6)
M_EXPECT = {
    "COO": dict(pos=[[0, 6], []], crd=[[0, 0, 2, 2, 2, 3], [1, 4, 0, 1, 5, 3]]),
    "CSR": dict(pos=[[4], [0, 2, 2, 5, 6]], crd=[[], [1, 4, 0, 1, 5, 3]]),
    "DCSR": dict(pos=[[0, 3], [0, 2, 5, 6]], crd=[[0, 2, 3], [1, 4, 0, 1, 5, 3]]),
}
# a 3x3x4 tensor
T_COORDS = ([0, 0, 0, 2, 2, 2, 2], [0, 0, 2, 1, 1, 2, 2], [1, 3, 0, 1, 2, 0, 3])
T_VAL = [1.0, 2.0, 3.0, 4.0, 5.0, 6.0, 7.0]
T_DIMS = (3, 3, 4)
T_CSF = dict(pos=[[0, 2], [0, 2, 4], [0, 2, 3, 5, 7]], crd=[[0, 2], [0, 2, 1, 2], [1, 3, 0, 1, 2, 0, 3]])


@pytest.mark.parametrize("fmt", list(FORMATS_2D))
def test_worked_matrix(fmt):
    rng = np.random.default_rng(0)
    p = rng.permutation(6)                                  # feed the entries in arbitrary order
    coords = [np.array(c)[p] for c in M_COORDS]
    pk = oracle.pack(coords, np.array(M_VAL)[p], M_DIMS, (0, 1), FORMATS_2D[fmt])
    for l in range(2):
        assert pk.pos[l].tolist() == M_EXPECT[fmt]["pos"][l]
        assert pk.crd[l].tolist() == M_EXPECT[fmt]["crd"][l]
    assert pk.val.tolist() == M_VAL
    assert p[pk.perm].tolist() == list(range(6))


def test_worked_tensor_csf_and_coo():
    p = np.random.default_rng(1).permutation(7)
    coords = [np.array(c)[p] for c in T_COORDS]
    pk = oracle.pack(coords, np.array(T_VAL)[p], T_DIMS, (0, 1, 2), (CU, CU, CU))
    for l in range(3):
        assert pk.pos[l].tolist() == T_CSF["pos"][l]
        assert pk.crd[l].tolist() == T_CSF["crd"][l]
    assert pk.val.tolist() == T_VAL
    coo = oracle.pack(coords, np.array(T_VAL)[p], T_DIMS, (0, 1, 2), (CN, S, S))
    assert coo.pos[0].tolist() == [0, 7] and coo.pos[1].size == 0 and coo.pos[2].size == 0
    for l in range(3):
        assert coo.crd[l].tolist() == list(T_COORDS[l])


def _check_layout(coords, val, dims, mode_order, attr):
    pk = oracle.pack(coords, val, dims, mode_order, attr)
    want_c, want_v = _sorted_entries(coords, val, mode_order)
    got = enumerate_entries(attr, pk.pos, pk.crd)
    # Table 1's loops enumerate exactly the input coordinate set, each once, in lexicographic order,
    # and leaf positions run 0..nnz-1 in that order.
    assert [c for _, c in got] == want_c
    assert [m for m, _ in got] == list(range(len(want_c)))
    assert np.array_equal(pk.val.view(np.int64), want_v.view(np.int64))
    nnz = len(want_c)
    parents = 1
    for l, a in enumerate(attr):
        dim = dims[mode_order[l]]
        pos, crd = pk.pos[l], pk.crd[l]
        if a == D:
            assert pos.tolist() == [dim] and crd.size == 0
            parents *= dim
        elif a == CU:
            assert len(pos) == parents + 1 and pos[0] == 0 and pos[-1] == len(crd)
            assert np.all(np.diff(pos) >= 0)
            for q in range(parents):
                seg = crd[pos[q]:pos[q + 1]]
                assert np.all(np.diff(seg) > 0)             # strictly ascending inside a parent
            parents = len(crd)
        elif a == CN:
            assert pos.tolist() == [0, nnz] and len(crd) == nnz
            parents = nnz
        else:
            assert pos.size == 0 and len(crd) == parents
        if crd.size:
            assert crd.min() >= 0 and crd.max() < dim
    assert parents == nnz
    return pk


@pytest.mark.parametrize("fmt", list(FORMATS_2D))
@pytest.mark.parametrize("dims,nnz,seed", [((7, 5), 12, 1), ((1, 9), 4, 2), ((9, 1), 4, 3), ((6, 6), 36, 4),
                                           ((8, 8), 1, 5), ((8, 8), 0, 6), ((40, 30), 200, 7)])
def test_table1_loops_2d(fmt, dims, nnz, seed):
    coords, val = synth.random_coo(dims, nnz, seed)
    _check_layout(_np(coords), val.numpy(), dims, (0, 1), FORMATS_2D[fmt])
    _check_layout(_np(coords), val.numpy(), dims, (1, 0), FORMATS_2D[fmt])     # column-major storage order


@pytest.mark.parametrize("fmt", list(FORMATS_3D))
@pytest.mark.parametrize("mode_order", [(0, 1, 2), (1, 0, 2), (2, 1, 0), (1, 2, 0)])
@pytest.mark.parametrize("dims,nnz,seed", [((4, 5, 6), 30, 1), ((3, 1, 7), 9, 2), ((5, 5, 5), 125, 3),
                                           ((6, 4, 3), 0, 4), ((9, 8, 7), 1, 5), ((12, 10, 8), 150, 6)])
def test_table1_loops_3d(fmt, mode_order, dims, nnz, seed):
    coords, val = synth.random_coo(dims, nnz, seed)
    _check_layout(_np(coords), val.numpy(), dims, mode_order, FORMATS_3D[fmt])


def test_order4_csf():
    dims = (4, 3, 5, 2)
    coords, val = synth.random_coo(dims, 40, 11)
    _check_layout(_np(coords), val.numpy(), dims, (0, 1, 2, 3), (CU, CU, CU, CU))
    _check_layout(_np(coords), val.numpy(), dims, (3, 1, 0, 2), (CN, S, S, S))


@pytest.mark.parametrize("dims,nnz,seed", [((50, 40), 300, 1), ((200, 300), 5000, 2), ((64, 64), 64, 3)])
def test_csr_equals_scipy(dims, nnz, seed):
    coords, val = synth.random_coo(dims, nnz, seed)
    i, j = _np(coords)
    pk = oracle.pack([i, j], val.numpy(), dims, (0, 1), (D, CU))
    ref = sp.coo_matrix((val.numpy(), (i, j)), shape=dims).tocsr()
    ref.sort_indices()
    assert np.array_equal(pk.pos[1], ref.indptr)
    assert np.array_equal(pk.crd[1], ref.indices)
    assert np.array_equal(pk.val, ref.data)
    # DCSR = CSR with the empty rows squeezed out
    dc = oracle.pack([i, j], val.numpy(), dims, (0, 1), (CU, CU))
    rows = np.flatnonzero(np.diff(ref.indptr))
    assert np.array_equal(dc.crd[0], rows) and dc.pos[0].tolist() == [0, len(rows)]
    assert np.array_equal(dc.pos[1], np.concatenate([ref.indptr[rows], [ref.nnz]]))
    assert np.array_equal(dc.crd[1], ref.indices)
    # CSC through mode_order
    pc = oracle.pack([i, j], val.numpy(), dims, (1, 0), (D, CU))
    refc = sp.coo_matrix((val.numpy(), (i, j)), shape=dims).tocsc()
    refc.sort_indices()
    assert np.array_equal(pc.pos[1], refc.indptr) and np.array_equal(pc.crd[1], refc.indices)
    assert np.array_equal(pc.val, refc.data)


def test_csf_upper_levels_are_dcsr_of_projection():
    dims = (30, 20, 25)
    coords, val = synth.random_coo(dims, 600, 5)
    i, j, k = _np(coords)
    csf = oracle.pack([i, j, k], val.numpy(), dims, (0, 1, 2), (CU, CU, CU))
    pairs = np.unique(np.stack([i, j], 1), axis=0)
    dc = oracle.pack([pairs[:, 0], pairs[:, 1]], np.ones(len(pairs)), dims[:2], (0, 1), (CU, CU))
    assert np.array_equal(csf.pos[0], dc.pos[0]) and np.array_equal(csf.crd[0], dc.crd[0])
    assert np.array_equal(csf.pos[1], dc.pos[1]) and np.array_equal(csf.crd[1], dc.crd[1])
    # all-ones closed form: the leaf pos differences are the fiber lengths
    _, counts = np.unique(i.astype(np.int64) * dims[1] + j, return_counts=True)
    assert np.array_equal(np.diff(csf.pos[2]), counts)


def test_shuffle_invariance():
    dims = (15, 14, 13)
    coords, val = synth.random_coo(dims, 400, 9)
    c = _np(coords)
    a = oracle.pack(c, val.numpy(), dims, (0, 1, 2), (CU, CU, CU))
    p = np.random.default_rng(3).permutation(len(val))
    b = oracle.pack([x[p] for x in c], val.numpy()[p], dims, (0, 1, 2), (CU, CU, CU))
    for l in range(3):
        assert np.array_equal(a.pos[l], b.pos[l]) and np.array_equal(a.crd[l], b.crd[l])
    assert np.array_equal(a.val, b.val)
    assert np.array_equal(p[b.perm], a.perm)


def test_rejects_bad_input():
    with pytest.raises(oracle.OracleError) as e:
        oracle.pack([[0, 0], [1, 1]], [1.0, 2.0], (2, 2), (0, 1), (D, CU))
    assert e.value.code == -4
    with pytest.raises(oracle.OracleError) as e:
        oracle.pack([[0, 0], [1, 1]], [1.0, 2.0], (2, 2), (0, 1), (CN, S))
    assert e.value.code == -4
    with pytest.raises(oracle.OracleError) as e:
        oracle.pack([[0, 2], [1, 1]], [1.0, 2.0], (2, 2), (0, 1), (D, CU))
    assert e.value.code == -3
    for bad in [(CU, D), (CU, CN), (CU, S), (S, S), (D, D)]:
        with pytest.raises(oracle.OracleError) as e:
            oracle.pack([[0], [1]], [1.0], (2, 2), (0, 1), bad)
        assert e.value.code == -2
    with pytest.raises(oracle.OracleError):
        oracle.pack([[0], [1]], [1.0], (2, 2), (0, 0), (D, CU))


# ----------------------------------------------------------------------------- merging duplicates
def test_sum_duplicates_against_a_dictionary_and_scipy():
    import scipy.sparse as sp
    rng = np.random.default_rng(5)
    dims = (7, 9)
    n = 300                                            # 63 cells: many duplicates
    ci, cj = rng.integers(0, 7, n).astype(np.int32), rng.integers(0, 9, n).astype(np.int32)
    v = rng.integers(-4, 5, n).astype(np.float64)      # small integers: every order of summation is exact
    (oi, oj), ov, first = oracle.sum_duplicates([ci, cj], v, dims, (0, 1))
    acc, seen_first = {}, {}
    for e in range(n):
        acc[(ci[e], cj[e])] = acc.get((ci[e], cj[e]), 0.0) + v[e]
        seen_first.setdefault((ci[e], cj[e]), e)
    cells = sorted(acc)
    assert list(zip(oi.tolist(), oj.tolist())) == cells
    assert ov.tolist() == [acc[k] for k in cells] and first.tolist() == [seen_first[k] for k in cells]
    csr = sp.coo_matrix((v, (ci, cj)), shape=dims).tocsr()      # scipy sums duplicates on conversion
    csr.sort_indices()
    pk = oracle.pack([ci, cj], v, dims, (0, 1), (oracle.D, oracle.CU), sum_duplicates_first=True)
    assert pk.pos[1].tolist() == csr.indptr.tolist() and pk.crd[1].tolist() == csr.indices.tolist()
    assert pk.val.tolist() == csr.data.tolist()
    # column-major storage order merges the same cells
    (pi, pj), pv, _ = oracle.sum_duplicates([ci, cj], v, dims, (1, 0))
    assert sorted(zip(pi.tolist(), pj.tolist())) == cells
    assert sorted(zip(pi.tolist(), pj.tolist(), pv.tolist())) == sorted((a, b, acc[(a, b)]) for a, b in cells)


def test_sum_duplicates_adds_in_input_order():
    # 1e16 + 1 + 1 differs from 1 + 1 + 1e16 in double: the sum must follow the order the entries were given
    c = [np.array([2, 2, 2, 0], dtype=np.int32), np.array([1, 1, 1, 0], dtype=np.int32), np.array([3, 3, 3, 0], dtype=np.int32)]
    _, v1, _ = oracle.sum_duplicates(c, np.array([1e16, 1.0, 1.0, 5.0]), (3, 2, 4), (0, 1, 2))
    _, v2, _ = oracle.sum_duplicates(c, np.array([1.0, 1.0, 1e16, 5.0]), (3, 2, 4), (0, 1, 2))
    assert v1.tolist() == [5.0, (1e16 + 1.0) + 1.0] and v2.tolist() == [5.0, (1.0 + 1.0) + 1e16] and v1[1] != v2[1]


def test_without_the_flag_duplicates_are_still_rejected():
    c = [np.array([1, 1], dtype=np.int32), np.array([2, 2], dtype=np.int32)]
    with pytest.raises(oracle.OracleError):
        oracle.pack(c, np.array([1.0, 2.0]), (3, 3), (0, 1), (oracle.D, oracle.CU))
    pk = oracle.pack(c, np.array([1.0, 2.0]), (3, 3), (0, 1), (oracle.D, oracle.CU), sum_duplicates_first=True)
    assert pk.val.tolist() == [3.0] and pk.crd[1].tolist() == [2] and pk.pos[1].tolist() == [0, 0, 1, 1]
