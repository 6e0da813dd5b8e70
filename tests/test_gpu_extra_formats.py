"""GPU parity of the ELLPACK format ([D,D,S]: packing, SpMV, SpMM) and of the element-wise sparse x dense
product, against the CPU oracle (oracle/extra.py for the packing and the product's values, the COO-loop oracle
for the contractions)."""
import numpy as np
import pytest
import torch

import oracle
import synth
from oracle import D, CU, CN, S
from oracle import extra

pytestmark = pytest.mark.gpu

comet = pytest.importorskip("paper_2102_05187_b200")
from gpu_util import assert_close, assert_equal_arrays, dev, upload_packed  # noqa: E402


@pytest.fixture(autouse=True)
def _need_gpu(cuda_device):
    yield


def _np(coords):
    return [c.numpy() for c in coords]


MATRICES = [((64, 48), 700, 1), ((300, 200), 5000, 2), ((1, 500), 300, 3), ((500, 1), 200, 4), ((40, 40), 1600, 5),
            ((200, 300), 1, 6), ((200, 300), 0, 7), ((3000, 100), 400, 8)]


@pytest.mark.parametrize("dims,nnz,seed", MATRICES)
@pytest.mark.parametrize("mode_order", [(0, 1), (1, 0)])
def test_ellpack_pack_is_bit_exact(dims, nnz, seed, mode_order):
    coords, val = synth.random_coo(dims, nnz, seed)
    want = extra.pack_ellpack(_np(coords), val.numpy(), dims, mode_order)
    got = comet.pack([c.cuda() for c in coords], val.cuda(), dims, mode_order, (D, S))
    assert got.attr == (D, D, S) and got.mode_order == want.mode_order and got.dims == want.dims
    assert got.nnz == want.val.size
    assert_equal_arrays(got.pos(0), want.pos[0], "pos0")
    assert_equal_arrays(got.pos(1), want.pos[1], "pos1")
    assert_equal_arrays(got.crd(2), want.crd[2], "slot columns")
    assert_equal_arrays(got.val, want.val, "slot values")


@pytest.mark.parametrize("dims,nnz,seed", MATRICES)
@pytest.mark.parametrize("R", [1, 3, 16, 64])
def test_ellpack_products(dims, nnz, seed, R):
    coords, val = synth.random_coo(dims, nnz, seed)
    c, v = _np(coords), val.numpy()
    A = upload_packed(extra.pack_ellpack(c, v, dims))             # caller-built descriptor from the oracle's arrays
    x = synth.random_dense((dims[1],), seed).numpy()
    want, norm = oracle.spmv(c, v, dims, x)
    y = torch.full((dims[0],), float("nan"), dtype=torch.float64, device="cuda")
    comet.spmv(A, dev(x), y)
    assert_close(y, want, norm, what="ellpack spmv")
    B = synth.random_dense((dims[1], R), seed).numpy()
    want, norm = oracle.spmm(c, v, dims, B)
    C = torch.full((dims[0], R), float("nan"), dtype=torch.float64, device="cuda")
    comet.spmm(A, dev(B), C)
    assert_close(C, want, norm, what=f"ellpack spmm R={R}")


def test_ellpack_skips_padding_even_next_to_infinities():
    """Padding slots must not touch the operand: an infinite x[0] or B[0, :] may only reach rows that store column 0."""
    c = ([0, 0, 2], [1, 2, 0])
    v = [1.0, 2.0, 3.0]
    A = upload_packed(extra.pack_ellpack(c, v, (3, 3)))
    x = torch.tensor([float("inf"), 1.0, 1.0], dtype=torch.float64, device="cuda")
    y = comet.spmv(A, x)
    assert y.tolist() == [3.0, 0.0, float("inf")]
    C = comet.spmm(A, torch.stack([x, x], dim=1).contiguous())
    assert C[:, 0].tolist() == [3.0, 0.0, float("inf")]


def test_ellpack_scaled_workload_fp32_and_fp64():
    case = synth.make(1, scale=1.0)                               # uniform rows: the shape ELLPACK is meant for
    c, v = _np(case.coords), case.val.numpy()
    x = case.dense["x"].numpy()
    want, norm = oracle.spmv(c, v, case.dims, x)
    A = comet.pack([t.cuda() for t in case.coords], case.val.cuda(), case.dims, (0, 1), (D, S))
    assert_close(comet.spmv(A, dev(x)), want, norm, what="ellpack spmv C1")
    A32 = comet.pack([t.cuda() for t in case.coords], case.val.float().cuda(), case.dims, (0, 1), (D, S))
    v32 = case.val.float().double().numpy()
    x32 = case.dense["x"].float()
    want, norm = oracle.spmv(c, v32, case.dims, x32.double().numpy())
    assert_close(comet.spmv(A32, x32.cuda()).double(), want, norm, tol=1e-5, what="ellpack spmv C1 fp32")


FORMATS = [((30, 40), (0, 1), (D, CU)), ((30, 40), (1, 0), (D, CU)), ((30, 40), (0, 1), (CU, CU)), ((30, 40), (0, 1), (CN, S)),
           ((12, 9, 14), (0, 1, 2), (CU, CU, CU)), ((12, 9, 14), (2, 0, 1), (CU, CU, CU)), ((12, 9, 14), (0, 1, 2), (CN, S, S)),
           ((12, 9, 14), (1, 2, 0), (D, CU, CU)), ((5, 6, 4, 7), (0, 1, 2, 3), (CU, CU, CU, CU)),
           ((5, 6, 4, 7), (3, 1, 0, 2), (CN, S, S, S))]


@pytest.mark.parametrize("dims,mode_order,attr", FORMATS)
def test_elementwise_product(dims, mode_order, attr):
    nnz = int(np.prod(dims)) // 3
    coords, val = synth.random_coo(dims, nnz, 31)
    c, v = _np(coords), val.numpy()
    B = synth.random_dense(dims, 31).numpy()
    want, norm = extra.elementwise(c, v, dims, B)                 # per input entry
    pk = oracle.pack(c, v, dims, mode_order, attr)
    A = upload_packed(pk)
    Cs = comet.elementwise_mul(A, dev(B))
    assert Cs.attr == attr and Cs.nnz == A.nnz
    assert_close(Cs.val, want[pk.perm], norm[pk.perm], what="elementwise product")     # leaf position p holds input entry perm[p]
    # a strided view of B (its transpose made contiguous, then viewed back) gives the same numbers
    Bt = dev(B).permute(*reversed(range(len(dims)))).contiguous().permute(*reversed(range(len(dims))))
    assert torch.equal(comet.elementwise_mul(A, Bt).val, Cs.val)


def test_elementwise_product_on_ellpack_and_on_an_empty_tensor():
    dims = (30, 40)
    coords, val = synth.random_coo(dims, 300, 32)
    c, v = _np(coords), val.numpy()
    B = synth.random_dense(dims, 32).numpy()
    want, norm = extra.elementwise(c, v, dims, B)
    pk = extra.pack_ellpack(c, v, dims)
    Cs = comet.elementwise_mul(upload_packed(pk), dev(B))
    keep = pk.perm >= 0
    got = Cs.val.cpu().numpy()
    assert_close(got[keep], want[pk.perm[keep]], norm[pk.perm[keep]], what="elementwise on ellpack")
    assert not got[~keep].any()
    empty = upload_packed(oracle.pack([np.zeros(0, np.int32)] * 2, np.zeros(0), dims, (0, 1), (D, CU)))
    assert comet.elementwise_mul(empty, dev(B)).nnz == 0
