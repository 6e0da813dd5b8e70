"""GPU parity of comet_reorder: the new numbers of every mode must equal the CPU oracle's, integer for
integer; applying them must leave a contraction unchanged up to the relabelling."""
import numpy as np
import pytest
import torch

import oracle
import synth
from oracle import D, CU
from oracle.reorder import reorder as oracle_reorder, window_columns

pytestmark = pytest.mark.gpu

comet = pytest.importorskip("paper_2102_05187_b200")
from gpu_util import assert_close, dev  # noqa: E402


@pytest.fixture(autouse=True)
def _need_gpu(cuda_device):
    yield


def _check(coords, dims, iterations):
    want = oracle_reorder([c.numpy() for c in coords], dims, iterations)
    got = comet.reorder([c.cuda() for c in coords], dims, iterations)
    for m in range(len(dims)):
        assert got[m].dtype == torch.int32 and got[m].cpu().numpy().tolist() == want[m].tolist(), f"mode {m}"
    return got


@pytest.mark.parametrize("dims,nnz,seed", [((7, 5), 12, 1), ((1, 9), 4, 2), ((40, 30), 300, 3), ((300, 200), 5000, 4),
                                           ((50, 50), 0, 5), ((20, 18, 16), 900, 6), ((1, 30, 30), 300, 7),
                                           ((2000, 5, 7), 500, 8), ((3000, 100), 400, 9),
                                           ((9, 8, 7, 6), 400, 10), ((40, 3, 1, 25), 600, 11)])
@pytest.mark.parametrize("iterations", [0, 1, 2, 4])
def test_labels_equal_the_oracle(dims, nnz, seed, iterations):
    coords, _ = synth.random_coo(dims, nnz, seed)
    _check(coords, dims, iterations)


def test_duplicates_and_ties_follow_the_oracle():
    g = np.random.default_rng(3)
    dims = (9, 7)
    coords = [torch.from_numpy(g.integers(0, d, 500).astype(np.int32)) for d in dims]     # every cell many times
    _check(coords, dims, 3)
    dims3 = (5, 4, 3)
    coords3 = [torch.from_numpy(g.integers(0, d, 400).astype(np.int32)) for d in dims3]
    _check(coords3, dims3, 3)


def test_hidden_band_is_recovered_and_spmm_is_unchanged():
    g = np.random.default_rng(0)
    n, L, R = 6000, 8, 4
    ti = np.repeat(np.arange(n), L)
    tj = (ti + np.tile(np.arange(L), n)) % n
    rho, sig = g.permutation(n), g.permutation(n)
    r, c = rho[ti].astype(np.int32), sig[tj].astype(np.int32)
    v = g.standard_normal(n * L)
    B = g.standard_normal((n, R))
    lr, lc = comet.reorder([dev(r), dev(c)], (n, n), 5)
    want = oracle_reorder([r, c], (n, n), 5)
    assert lr.cpu().numpy().tolist() == want[0].tolist() and lc.cpu().numpy().tolist() == want[1].tolist()
    nr, nc = lr[dev(r).long()], lc[dev(c).long()]
    assert window_columns(nr.cpu().numpy(), nc.cpu().numpy(), n) < 1.35 * window_columns(ti, tj, n)
    # the product on the relabelled matrix, with the rows of B moved along, is the original product relabelled
    Y, norm = oracle.spmm([r, c], v, (n, n), B)
    A = comet.pack([nr.contiguous(), nc.contiguous()], dev(v), (n, n), (0, 1), (D, CU))
    Bp = torch.empty((n, R), dtype=torch.float64, device="cuda")
    Bp[lc.long()] = dev(B)
    Yp = comet.spmm(A, Bp)
    assert_close(Yp[lr.long()], Y, norm, what="spmm after reordering")


def test_bad_coordinates_and_orders_are_reported():
    with pytest.raises(comet.CometError) as e:
        comet.reorder([dev(np.array([0, 5], dtype=np.int32)), dev(np.array([0, 1], dtype=np.int32))], (3, 3), 2)
    assert comet.binding.STATUS_NAMES[e.value.status] == "COMET_ERR_COORD_OUT_OF_RANGE"
    with pytest.raises(comet.CometError) as e:
        comet.reorder([dev(np.zeros(2, dtype=np.int32))], (2,), 1)               # a vector has nothing to reorder by
    assert e.value.status == -2
