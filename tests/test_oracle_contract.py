"""Pins for the oracle's contractions: dense brute force written straight from the definitions
(numpy.einsum over a densified tiny tensor), library routines on unfoldings (scipy csr @ dense),
closed forms (all-ones -> counts, identity factors -> scatter, R=1 reductions), exact small-integer
cases, exact power-of-two linearity, and a hand-worked example."""
import numpy as np
import pytest
import scipy.sparse as sp

import oracle
import synth


def _np(coords):
    return [c.numpy() for c in coords]


def _dense(coords, val, dims):
    X = np.zeros(dims)
    X[tuple(coords)] = val
    return X


def _close(got, want, norm, tol=1e-13):
    assert got.shape == want.shape
    assert np.all(np.abs(got - want) <= tol * norm + 0.0), float(np.max(np.abs(got - want) - tol * norm))


# ----------------------------------------------------------------------------- hand-worked example
def test_worked_example():
    mc = ([0, 0, 2, 2, 2, 3], [1, 4, 0, 1, 5, 3])
    mv = [1.0, 2.0, 3.0, 4.0, 5.0, 6.0]
    y, _ = oracle.spmv(mc, mv, (4, 6), [1.0, 2, 3, 4, 5, 6])
    assert y.tolist() == [12.0, 0.0, 41.0, 24.0]
    Y, _ = oracle.spmm(mc, mv, (4, 6), np.arange(12.0).reshape(6, 2))
    assert Y.tolist() == [[18, 21], [0, 0], [58, 70], [36, 42]]
    tc = ([0, 0, 0, 2, 2, 2, 2], [0, 0, 2, 1, 1, 2, 2], [1, 3, 0, 1, 2, 0, 3])
    tv = [1.0, 2.0, 3.0, 4.0, 5.0, 6.0, 7.0]
    keys, y, _ = oracle.ttv(tc, tv, (3, 3, 4), 2, [1.0, 10, 100, 1000])
    assert keys.tolist() == [0, 2, 7, 8] and y.tolist() == [2010.0, 3.0, 540.0, 7006.0]
    keys, Y, _ = oracle.ttm(tc, tv, (3, 3, 4), 2, np.array([[1.0, 0], [0, 1], [1, 1], [2, -1]]))
    assert Y.tolist() == [[4, -1], [3, 0], [5, 9], [20, -7]]
    A, _ = oracle.mttkrp(tc, tv, (3, 3, 4), 0,
                         [None, np.array([[1.0, 2], [3, 4], [5, 6]]), np.array([[1.0, -1], [2, 0], [0, 1], [1, 1]])])
    assert A.tolist() == [[19, -14], [0, 0], [89, 26]]


# ----------------------------------------------------------------------------- dense brute force
@pytest.mark.parametrize("dims,nnz,seed", [((8, 7), 20, 1), ((1, 5), 3, 2), ((6, 1), 4, 3), ((5, 5), 25, 4),
                                           ((7, 6), 0, 5)])
@pytest.mark.parametrize("integer", [False, True])
def test_matrix_ops_vs_einsum(dims, nnz, seed, integer):
    coords, val = synth.random_coo(dims, nnz, seed, integer_values=integer)
    c, v = _np(coords), val.numpy()
    X = _dense(c, v, dims)
    x = synth.random_dense((dims[1],), seed, 51, integer_values=integer).numpy()
    B = synth.random_dense((dims[1], 3), seed, 52, integer_values=integer).numpy()
    y, yn = oracle.spmv(c, v, dims, x)
    Y, Yn = oracle.spmm(c, v, dims, B)
    if integer:
        assert np.array_equal(y, np.einsum("ij,j->i", X, x)) and np.array_equal(Y, np.einsum("ij,jr->ir", X, B))
    else:
        _close(y, np.einsum("ij,j->i", X, x), yn)
        _close(Y, np.einsum("ij,jr->ir", X, B), Yn)
    _close(yn, np.einsum("ij,j->i", np.abs(X), np.abs(x)), yn)
    _close(Yn, np.einsum("ij,jr->ir", np.abs(X), np.abs(B)), Yn)


EIN_TTV = {0: "ijk,i->jk", 1: "ijk,j->ik", 2: "ijk,k->ij"}
EIN_TTM = {0: "ijk,ir->jkr", 1: "ijk,jr->ikr", 2: "ijk,kr->ijr"}
EIN_MTTKRP = {0: "ijk,jr,kr->ir", 1: "ijk,ir,kr->jr", 2: "ijk,ir,jr->kr"}


@pytest.mark.parametrize("dims,nnz,seed", [((8, 7, 6), 40, 1), ((3, 1, 5), 7, 2), ((4, 4, 4), 64, 3),
                                           ((5, 6, 7), 0, 4), ((6, 5, 4), 1, 5)])
@pytest.mark.parametrize("mode", [0, 1, 2])
@pytest.mark.parametrize("integer", [False, True])
def test_tensor_ops_vs_einsum(dims, nnz, seed, mode, integer):
    coords, val = synth.random_coo(dims, nnz, seed, integer_values=integer)
    c, v = _np(coords), val.numpy()
    X = _dense(c, v, dims)
    R = 3
    vec = synth.random_dense((dims[mode],), seed, 51, integer_values=integer).numpy()
    U = synth.random_dense((dims[mode], R), seed, 52, integer_values=integer).numpy()
    F = [synth.random_dense((d, R), seed, 60 + m, integer_values=integer).numpy() for m, d in enumerate(dims)]
    kept = [m for m in range(3) if m != mode]
    keys, y, yn = oracle.ttv(c, v, dims, mode, vec)
    _, Y, Yn = oracle.ttm(c, v, dims, mode, U)
    A, An = oracle.mttkrp(c, v, dims, mode, F)
    ka, kb = keys // dims[kept[1]], keys % dims[kept[1]]
    # the stored fibers are exactly the (a,b) pairs that hold an entry, in lexicographic order
    pairs = np.unique(np.stack([c[kept[0]], c[kept[1]]], 1), axis=0) if nnz else np.zeros((0, 2), dtype=np.int64)
    assert np.array_equal(np.stack([ka, kb], 1), pairs)
    dy = np.einsum(EIN_TTV[mode], X, vec)
    dY = np.einsum(EIN_TTM[mode], X, U)
    others = [F[m] for m in kept]
    dA = np.einsum(EIN_MTTKRP[mode], X, *others)
    if integer:
        assert np.array_equal(y, dy[ka, kb]) and np.array_equal(Y, dY[ka, kb]) and np.array_equal(A, dA)
    else:
        _close(y, dy[ka, kb], yn)
        _close(Y, dY[ka, kb], Yn)
        _close(A, dA, An)
    # everything outside the stored fibers is structurally zero in the dense result
    mask = np.ones(dy.shape, bool)
    mask[ka, kb] = False
    assert np.all(dy[mask] == 0)
    _close(An, np.einsum(EIN_MTTKRP[mode], np.abs(X), *[np.abs(f) for f in others]), An)


# ----------------------------------------------------------------------------- library routines
@pytest.mark.parametrize("dims,nnz,seed", [((300, 200), 4000, 1), ((1000, 50), 3000, 2)])
def test_spmm_vs_scipy(dims, nnz, seed):
    coords, val = synth.random_coo(dims, nnz, seed)
    i, j = _np(coords)
    A = sp.coo_matrix((val.numpy(), (i, j)), shape=dims).tocsr()
    B = synth.random_dense((dims[1], 16), seed).numpy()
    Y, Yn = oracle.spmm([i, j], val.numpy(), dims, B)
    _close(Y, A @ B, Yn)
    y, yn = oracle.spmv([i, j], val.numpy(), dims, B[:, 0])
    _close(y, A @ B[:, 0], yn)
    _close(Y[:, :1], y[:, None], Yn[:, :1], tol=0)           # SpMM with R = 1 is SpMV, term for term
    # sampled rows agree with the full evaluation bit for bit
    rows = np.array([0, 5, 17, dims[0] - 1])
    Ys, _ = oracle.spmm([i, j], val.numpy(), dims, B, rows=rows)
    assert np.array_equal(Ys, Y[rows])


@pytest.mark.parametrize("mode", [0, 1, 2])
def test_tensor_ops_vs_unfolding(mode):
    dims = (40, 30, 20)
    coords, val = synth.random_coo(dims, 3000, 7)
    c, v = _np(coords), val.numpy()
    R = 8
    kept = [m for m in range(3) if m != mode]
    # TTV / TTM = SpMV / SpMM on the mode-n unfolding (rows = kept pairs, columns = contracted index)
    rows = c[kept[0]].astype(np.int64) * dims[kept[1]] + c[kept[1]]
    Xn = sp.coo_matrix((v, (rows, c[mode])), shape=(dims[kept[0]] * dims[kept[1]], dims[mode])).tocsr()
    U = synth.random_dense((dims[mode], R), 3).numpy()
    keys, Y, Yn = oracle.ttm(c, v, dims, mode, U)
    _close(Y, (Xn @ U)[keys], Yn)
    _, y, yn = oracle.ttv(c, v, dims, mode, U[:, 0])
    _close(y, (Xn @ U[:, 0])[keys], yn)
    _close(Y[:, 0], y, yn, tol=0)                            # TTM with R = 1 column is TTV
    # MTTKRP = X_(n) (Q khatri-rao P): unfolding columns p + q * dim_p for kept modes p < q
    F = [synth.random_dense((d, R), 4, 60 + m).numpy() for m, d in enumerate(dims)]
    P, Q = F[kept[0]], F[kept[1]]
    KR = (Q[:, None, :] * P[None, :, :]).reshape(dims[kept[0]] * dims[kept[1]], R)
    cols = c[kept[0]].astype(np.int64) + c[kept[1]].astype(np.int64) * dims[kept[0]]
    Xm = sp.coo_matrix((v, (c[mode], cols)), shape=(dims[mode], dims[kept[0]] * dims[kept[1]])).tocsr()
    A, An = oracle.mttkrp(c, v, dims, mode, F)
    _close(A, Xm @ KR, An)
    sample = np.array([1, 3, dims[mode] - 1])
    As, _ = oracle.mttkrp(c, v, dims, mode, F, rows=sample)
    assert np.array_equal(As, A[sample])
    ks = keys[::7]
    _, Ys, _ = oracle.ttm(c, v, dims, mode, U, keys=ks)
    assert np.array_equal(Ys, Y[::7])


# ----------------------------------------------------------------------------- closed forms
def test_all_ones_give_counts():
    dims = (25, 20, 15)
    coords, _ = synth.random_coo(dims, 900, 13)
    c = _np(coords)
    ones = np.ones(len(c[0]))
    # matrix view of the first two modes is not distinct, so use a matrix case of its own
    mc, _ = synth.random_coo((60, 50), 700, 14)
    mi, mj = _np(mc)
    Y, Yn = oracle.spmm([mi, mj], np.ones(len(mi)), (60, 50), np.ones((50, 4)))
    counts = np.bincount(mi, minlength=60)
    assert np.array_equal(Y, np.repeat(counts[:, None], 4, 1)) and np.array_equal(Yn, Y)
    csr = oracle.pack([mi, mj], np.ones(len(mi)), (60, 50), (0, 1), (oracle.D, oracle.CU))
    assert np.array_equal(np.diff(csr.pos[1]), counts)       # row counts = pos differences
    keys, y, _ = oracle.ttv(c, ones, dims, 2, np.ones(dims[2]))
    csf = oracle.pack(c, ones, dims, (0, 1, 2), (oracle.CU,) * 3)
    assert np.array_equal(y, np.diff(csf.pos[2]))            # fiber lengths
    A, _ = oracle.mttkrp(c, ones, dims, 0, [None, np.ones((dims[1], 5)), np.ones((dims[2], 5))])
    assert np.array_equal(A, np.repeat(np.bincount(c[0], minlength=dims[0])[:, None], 5, 1))   # slice counts
    v = synth.random_dense((len(ones),), 15).numpy()
    A, An = oracle.mttkrp(c, v, dims, 0, [None, np.ones((dims[1], 2)), np.ones((dims[2], 2))])
    sums = np.zeros(dims[0])
    np.add.at(sums, c[0], v)
    _close(A[:, 0], sums, An[:, 0])                          # all-ones factors give the mode sums


def test_identity_factors_scatter():
    dims = (6, 5, 4)
    coords, val = synth.random_coo(dims, 50, 21)
    c, v = _np(coords), val.numpy()
    X = _dense(c, v, dims)
    keys, Y, _ = oracle.ttm(c, v, dims, 2, np.eye(dims[2]))
    assert np.array_equal(Y, X.reshape(-1, dims[2])[keys])   # U = I returns the fibers themselves
    mc, mv = synth.random_coo((7, 6), 20, 22)
    mi, mj = _np(mc)
    Y, _ = oracle.spmm([mi, mj], mv.numpy(), (7, 6), np.eye(6))
    assert np.array_equal(Y, _dense([mi, mj], mv.numpy(), (7, 6)))


def test_power_of_two_linearity_is_exact():
    dims = (30, 25, 20)
    coords, val = synth.random_coo(dims, 800, 31)
    c, v = _np(coords), val.numpy()
    F = [synth.random_dense((d, 4), 32, 60 + m).numpy() for m, d in enumerate(dims)]
    A, _ = oracle.mttkrp(c, v, dims, 0, F)
    A4, _ = oracle.mttkrp(c, 4.0 * v, dims, 0, F)
    assert np.array_equal(A4, 4.0 * A)
    _, Y, _ = oracle.ttm(c, v, dims, 2, F[2])
    _, Yh, _ = oracle.ttm(c, 0.5 * v, dims, 2, F[2])
    assert np.array_equal(Yh, 0.5 * Y)


def test_mode2_mttkrp_is_mode1_of_transposed_tensor():
    dims = (12, 11, 10)
    coords, val = synth.random_coo(dims, 300, 41)
    c, v = _np(coords), val.numpy()
    F = [synth.random_dense((d, 3), 42, 60 + m).numpy() for m, d in enumerate(dims)]
    A, _ = oracle.mttkrp(c, v, dims, 1, F)
    At, _ = oracle.mttkrp([c[1], c[0], c[2]], v, (dims[1], dims[0], dims[2]), 0, [F[1], F[0], F[2]])
    assert np.array_equal(A, At)


def test_input_order_does_not_matter_beyond_rounding():
    dims = (20, 20, 20)
    coords, val = synth.random_coo(dims, 2000, 51)
    c, v = _np(coords), val.numpy()
    F = [synth.random_dense((d, 4), 52, 60 + m).numpy() for m, d in enumerate(dims)]
    A, An = oracle.mttkrp(c, v, dims, 0, F)
    p = np.random.default_rng(5).permutation(len(v))
    Ap, _ = oracle.mttkrp([x[p] for x in c], v[p], dims, 0, F)
    _close(Ap, A, An, tol=2e-16)


def test_out_of_range_rejected():
    with pytest.raises(oracle.OracleError):
        oracle.spmv([[0], [9]], [1.0], (2, 2), [1.0, 1.0])
    with pytest.raises(oracle.OracleError):
        oracle.mttkrp([[0], [0], [5]], [1.0], (2, 2, 2), 0, [None, np.ones((2, 1)), np.ones((2, 1))])


# ----------------------------------------------------------------------------- order-N TTV / TTM
@pytest.mark.parametrize("dims,nnz,seed", [((5, 4, 3, 6), 120, 1), ((2, 7, 1, 5), 40, 2), ((3, 3, 3, 3), 81, 3),
                                           ((6, 5, 4), 70, 4), ((9, 7), 30, 5)])
@pytest.mark.parametrize("integer", [False, True])
def test_order_n_products_vs_einsum(dims, nnz, seed, integer):
    """The order-N oracle against numpy.einsum on the densified tensor, every mode, matrix and vector factor."""
    coords, val = synth.random_coo(dims, nnz, seed, integer_values=integer)
    c, v = _np(coords), val.numpy()
    X = _dense(c, v, dims)
    letters = "abcd"[:len(dims)]
    for mode in range(len(dims)):
        kept = [m for m in range(len(dims)) if m != mode]
        U = synth.random_dense((dims[mode], 3), seed, 40 + mode, integer_values=integer).numpy()
        keys, Y, norm = oracle.ttm_n(c, v, dims, mode, U)
        out = letters.replace(letters[mode], "") + "r"
        dense = np.einsum(f"{letters},{letters[mode]}r->{out}", X, U)
        dnorm = np.einsum(f"{letters},{letters[mode]}r->{out}", np.abs(X), np.abs(U))
        flat = dense.reshape(-1, 3)
        # the keys are exactly the kept-coordinate tuples that hold an entry, ascending
        occupied = np.unique(np.ravel_multi_index([c[m] for m in kept], [dims[m] for m in kept]))
        assert keys.tolist() == occupied.tolist()
        if integer:
            assert np.array_equal(Y, flat[keys])
        else:
            _close(Y, flat[keys], dnorm.reshape(-1, 3)[keys])
        _close(norm, dnorm.reshape(-1, 3)[keys], dnorm.reshape(-1, 3)[keys], tol=1e-14)
        mask = np.ones(flat.shape[0], dtype=bool)
        mask[keys] = False
        assert not flat[mask].any()                      # nothing outside the listed fibers
        # one column = the tensor-times-vector product
        _, y1, _ = oracle.ttm_n(c, v, dims, mode, U[:, 0].copy())
        assert np.array_equal(y1[:, 0], Y[:, 0])


@pytest.mark.parametrize("mode", [0, 1, 2])
def test_order_n_functions_agree_with_the_three_order_ones(mode):
    dims = (9, 8, 7)
    coords, val = synth.random_coo(dims, 200, 12)
    c, v = _np(coords), val.numpy()
    U = synth.random_dense((dims[mode], 4), 12).numpy()
    k3, Y3, n3 = oracle.ttm(c, v, dims, mode, U)
    kn, Yn, nn = oracle.ttm_n(c, v, dims, mode, U)
    assert k3.tolist() == kn.tolist() and np.array_equal(Y3, Yn) and np.array_equal(n3, nn)
    _, y3, _ = oracle.ttv(c, v, dims, mode, U[:, 1].copy())
    _, yn, _ = oracle.ttm_n(c, v, dims, mode, U[:, 1].copy())
    assert np.array_equal(y3, yn[:, 0])


def test_order_n_matrix_case_is_spmm():
    dims = (11, 13)
    coords, val = synth.random_coo(dims, 60, 8)
    c, v = _np(coords), val.numpy()
    B = synth.random_dense((13, 5), 8).numpy()
    Y, _ = oracle.spmm(c, v, dims, B)
    keys, Yn, _ = oracle.ttm_n(c, v, dims, 1, B)           # contracting the column mode of a matrix
    assert np.array_equal(Y[keys], Yn) and not np.delete(Y, keys, axis=0).any()


@pytest.mark.parametrize("dims,nnz,seed", [((5, 4, 3, 6), 120, 1), ((2, 7, 1, 5), 40, 2), ((3, 3, 3, 3), 81, 3),
                                           ((6, 5, 4), 70, 4)])
@pytest.mark.parametrize("integer", [False, True])
def test_order_n_mttkrp_vs_einsum(dims, nnz, seed, integer):
    coords, val = synth.random_coo(dims, nnz, seed, integer_values=integer)
    c, v = _np(coords), val.numpy()
    X = _dense(c, v, dims)
    R = 3
    F = [synth.random_dense((d, R), seed, 60 + m, integer_values=integer).numpy() for m, d in enumerate(dims)]
    letters = "abcd"[:len(dims)]
    for mode in range(len(dims)):
        others = [m for m in range(len(dims)) if m != mode]
        expr = letters + "," + ",".join(letters[m] + "r" for m in others) + "->" + letters[mode] + "r"
        want = np.einsum(expr, X, *[F[m] for m in others])
        norm = np.einsum(expr, np.abs(X), *[np.abs(F[m]) for m in others])
        got, gnorm = oracle.mttkrp_n(c, v, dims, mode, F)
        if integer:
            assert np.array_equal(got, want)
        else:
            _close(got, want, norm)
        _close(gnorm, norm, norm, tol=1e-14)
        rows = np.array(sorted({0, dims[mode] - 1, dims[mode] // 2}))
        sub, _ = oracle.mttkrp_n(c, v, dims, mode, F, rows=rows)
        assert np.array_equal(sub, got[rows])


@pytest.mark.parametrize("mode", [0, 1, 2])
def test_order_n_mttkrp_is_the_three_order_function_on_three_order_input(mode):
    dims = (9, 8, 7)
    coords, val = synth.random_coo(dims, 200, 12)
    c, v = _np(coords), val.numpy()
    F = [synth.random_dense((d, 5), 12, 60 + m).numpy() for m, d in enumerate(dims)]
    a3, n3 = oracle.mttkrp(c, v, dims, mode, F)
    an, nn = oracle.mttkrp_n(c, v, dims, mode, F)
    assert np.array_equal(a3, an) and np.array_equal(n3, nn)


def test_timed_baseline_agrees_with_the_parity_oracle():
    """The benchmark's timed CPU loop (double accumulators, 1 and several threads) against the long-double oracle."""
    from oracle import timed_baseline
    dims, R = (300, 200), 16
    coords, val = synth.random_coo(dims, 5000, 21)
    c, v = [x.numpy() for x in coords], val.numpy()
    B = synth.random_dense((dims[1], R), 21).numpy()
    want, norm = oracle.spmm(c, v, dims, B)
    for threads in (1, 3):
        got = timed_baseline.spmm(c, v, dims, B, threads)
        assert np.all(np.abs(got - want) <= 1e-12 * norm)
    assert timed_baseline.host_threads() >= 1
