"""Pins for the reordering oracle: it must return permutations, leave contractions unchanged up to the
relabelling, keep a matrix that is already in staircase order where it is, follow a tiny example worked by
hand, and recover a band hidden by random relabelling (the effect the paper's section describes)."""
import numpy as np

import oracle
import synth
from oracle.reorder import reorder, window_columns


def test_worked_example():
    # 3 x 4 matrix, entries (row, col): (0,3) (0,2) (1,0) (2,2) (2,1)
    r = np.array([0, 0, 1, 2, 2])
    c = np.array([3, 2, 0, 2, 1])
    # step for rows: smallest column of row 0 is 2, of row 1 is 0, of row 2 is 1  ->  order 1, 2, 0
    # so row 1 -> 0, row 2 -> 1, row 0 -> 2.
    # step for columns (rows renumbered): column 0 is touched by row 0 (old 1); column 1 by row 1 (old 2);
    # column 2 by rows 2 and 1 -> smallest 1; column 3 by row 2 -> order: col 0 (0), col 1 (1), col 2 (1), col 3 (2)
    rows, cols = reorder([r, c], (3, 4), 1)
    assert rows.tolist() == [2, 0, 1] and cols.tolist() == [0, 1, 2, 3]
    # an index without entries keeps its place behind the others
    rows, cols = reorder([r, c], (5, 4), 1)
    assert rows.tolist() == [2, 0, 1, 3, 4]


def test_result_is_a_permutation_and_zero_iterations_is_the_identity():
    g = np.random.default_rng(1)
    dims = (30, 20, 10)
    coords = [g.integers(0, d, 200) for d in dims]
    for it in (0, 1, 3):
        labels = reorder(coords, dims, it)
        for m, d in enumerate(dims):
            assert sorted(labels[m].tolist()) == list(range(d))
            if it == 0:
                assert labels[m].tolist() == list(range(d))


def test_contractions_are_unchanged_up_to_the_relabelling():
    g = np.random.default_rng(2)
    dims = (40, 30)
    cells = g.choice(dims[0] * dims[1], 300, replace=False)
    r, c = cells // dims[1], cells % dims[1]
    v = g.standard_normal(300)
    B = g.standard_normal((dims[1], 3))
    Y, _ = oracle.spmm([r, c], v, dims, B)
    lr, lc = reorder([r, c], dims, 2)
    Bp = np.empty_like(B)
    Bp[lc] = B                                        # row j of B moves to row new_label[j]
    Yp, _ = oracle.spmm([lr[r], lc[c]], v, dims, Bp)
    assert np.allclose(Yp[lr], Y, rtol=0, atol=1e-12)  # row i of the result moved to new_label[i]


def test_a_staircase_matrix_is_a_fixed_point():
    # rows whose smallest columns already ascend, columns whose smallest rows already ascend
    r = np.array([0, 0, 1, 1, 2, 3, 3])
    c = np.array([0, 1, 1, 2, 2, 3, 4])
    rows, cols = reorder([r, c], (4, 5), 3)
    assert rows.tolist() == [0, 1, 2, 3] and cols.tolist() == [0, 1, 2, 3, 4]


def test_a_hidden_band_is_recovered():
    g = np.random.default_rng(0)
    n, L = 1500, 8
    ti = np.repeat(np.arange(n), L)
    tj = (ti + np.tile(np.arange(L), n)) % n
    rho, sig = g.permutation(n), g.permutation(n)
    r, c = rho[ti], sig[tj]
    ideal = window_columns(ti, tj, n)
    before = window_columns(r, c, n)
    lr, lc = reorder([r, c], (n, n), 5)
    after = window_columns(lr[r], lc[c], n)
    assert before > 5 * ideal                         # the relabelling destroyed the locality ...
    assert after < 1.35 * ideal                       # ... and five iterations bring it back


def test_three_order_tensors_use_the_tuple_of_the_other_modes():
    # mode-0 indices 0 and 1 share their smallest mode-1 coordinate; the mode-2 coordinate decides
    c0 = np.array([0, 1, 2])
    c1 = np.array([1, 1, 0])
    c2 = np.array([5, 3, 9])
    l0, l1, l2 = reorder([c0, c1, c2], (3, 2, 10), 1)
    assert l0.tolist() == [2, 1, 0]                   # keys (1,5), (1,3), (0,9) -> order: index 2, index 1, index 0


def test_four_order_tensors_keep_the_contraction():
    """Order 4: the labels are permutations and an order-4 tensor-times-vector is unchanged up to the relabelling."""
    dims = (6, 5, 4, 7)
    coords, val = synth.random_coo(dims, 200, 12)
    c, v = [x.numpy() for x in coords], val.numpy()
    lab = reorder(c, dims, 3)
    for m, d in enumerate(dims):
        assert sorted(lab[m].tolist()) == list(range(d))
    x = synth.random_dense((dims[3],), 12).numpy()
    dense = np.zeros(dims)
    dense[tuple(c)] = v
    want = np.einsum("ijkl,l->ijk", dense, x)
    relabelled = np.zeros(dims)
    relabelled[tuple(lab[m][c[m]] for m in range(4))] = v
    xp = np.zeros_like(x)
    xp[lab[3]] = x
    got = np.einsum("ijkl,l->ijk", relabelled, xp)
    assert np.allclose(got[np.ix_(lab[0], lab[1], lab[2])], want, rtol=0, atol=1e-12)
