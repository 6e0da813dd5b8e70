"""GPU parity: every contraction of the CUDA library against the CPU oracle, element by element, on
the same seeded inputs. Structure arrays come from the oracle's packing here (caller-built
descriptors), so these tests isolate the contraction kernels; test_gpu_pack.py covers the packing."""
import numpy as np
import pytest
import torch

import oracle
import synth
from oracle import D, CU, CN, S

pytestmark = pytest.mark.gpu

comet = pytest.importorskip("paper_2102_05187_b200")
from gpu_util import FP64_TOL, assert_close, assert_equal_arrays, dev, upload_packed  # noqa: E402


def _np(coords):
    return [c.numpy() for c in coords]


@pytest.fixture(autouse=True)
def _need_gpu(cuda_device):
    yield


@pytest.fixture(params=[None, 8, 37])
def tile_items(request, monkeypatch):
    """Default tiling, and tiny / odd tiles so that segments straddle many tiles (carry path)."""
    if request.param is None:
        monkeypatch.delenv("COMET_TILE_ITEMS", raising=False)
    else:
        monkeypatch.setenv("COMET_TILE_ITEMS", str(request.param))
    return request.param


@pytest.fixture(params=["default", "resident", "stream", "stream-short-spans", "stream2", "stream2-short-spans"])
def seg_dot_path(request, monkeypatch):
    """SpMV/TTV kernel choice: the size-based default, then each large-input kernel forced on small inputs
    (the warp-stream kernel also with 128-entry spans, so that segments straddle many spans)."""
    monkeypatch.delenv("COMET_SEG_DOT_KERNEL", raising=False)
    monkeypatch.delenv("COMET_STREAM_SPAN", raising=False)
    if request.param == "resident":
        monkeypatch.setenv("COMET_SEG_DOT_KERNEL", "resident")
    elif request.param.startswith("stream"):
        monkeypatch.setenv("COMET_SEG_DOT_KERNEL", "stream2" if request.param.startswith("stream2") else "stream")
        if request.param.endswith("short-spans"):
            monkeypatch.setenv("COMET_STREAM_SPAN", "128")
    return request.param


def test_worked_example():
    mc = ([0, 0, 2, 2, 2, 3], [1, 4, 0, 1, 5, 3])
    mv = [1.0, 2.0, 3.0, 4.0, 5.0, 6.0]
    for attr in [(D, CU), (CU, CU), (CN, S)]:
        A = upload_packed(oracle.pack(mc, mv, (4, 6), (0, 1), attr))
        y = comet.spmv(A, dev([1.0, 2, 3, 4, 5, 6]))
        assert y.tolist() == [12.0, 0.0, 41.0, 24.0]
        Y = comet.spmm(A, dev(np.arange(12.0).reshape(6, 2)))
        assert Y.tolist() == [[18, 21], [0, 0], [58, 70], [36, 42]]
    tc = ([0, 0, 0, 2, 2, 2, 2], [0, 0, 2, 1, 1, 2, 2], [1, 3, 0, 1, 2, 0, 3])
    tv = [1.0, 2.0, 3.0, 4.0, 5.0, 6.0, 7.0]
    X = upload_packed(oracle.pack(tc, tv, (3, 3, 4), (0, 1, 2), (CU, CU, CU)))
    Y = comet.ttv(X, 2, dev([1.0, 10, 100, 1000]))
    assert Y.val.tolist() == [2010.0, 3.0, 540.0, 7006.0]
    assert Y.pos(1).tolist() == [0, 2, 2, 4] and Y.crd(1).tolist() == [0, 2, 1, 2] and Y.pos(0).tolist() == [3]
    Z = comet.ttm(X, 2, dev(np.array([[1.0, 0], [0, 1], [1, 1], [2, -1]])))
    assert Z.val.reshape(4, 2).tolist() == [[4, -1], [3, 0], [5, 9], [20, -7]]
    assert Z.attr == (CU, CU, D) and Z.dims == (3, 3, 2) and Z.pos(2).tolist() == [2]
    assert Z.crd(0).tolist() == [0, 2] and Z.pos(1).tolist() == [0, 2, 4] and Z.crd(1).tolist() == [0, 2, 1, 2]
    F = [None, dev(np.array([[1.0, 2], [3, 4], [5, 6]])), dev(np.array([[1.0, -1], [2, 0], [0, 1], [1, 1]]))]
    for attr in [(CU, CU, CU), (CN, S, S)]:
        X = upload_packed(oracle.pack(tc, tv, (3, 3, 4), (0, 1, 2), attr))
        assert comet.mttkrp(X, 0, F).tolist() == [[19, -14], [0, 0], [89, 26]]


MATRIX_CASES = [((64, 48), 700, 1), ((300, 200), 5000, 2), ((1, 500), 300, 3), ((500, 1), 200, 4),
                ((40, 40), 1600, 5), ((200, 300), 1, 6), ((200, 300), 0, 7), ((3000, 100), 400, 8)]


@pytest.mark.parametrize("dims,nnz,seed", MATRIX_CASES)
@pytest.mark.parametrize("attr", [(D, CU), (CU, CU), (CN, S)])
def test_spmv(dims, nnz, seed, attr, tile_items, seg_dot_path):
    coords, val = synth.random_coo(dims, nnz, seed)
    c, v = _np(coords), val.numpy()
    x = synth.random_dense((dims[1],), seed).numpy()
    want, norm = oracle.spmv(c, v, dims, x)
    A = upload_packed(oracle.pack(c, v, dims, (0, 1), attr))
    y = torch.full((dims[0],), float("nan"), dtype=torch.float64, device="cuda")   # every entry must be written
    comet.spmv(A, dev(x), y)
    assert_close(y, want, norm, what="spmv")


@pytest.mark.parametrize("dims,nnz,seed", MATRIX_CASES)
@pytest.mark.parametrize("attr", [(D, CU), (CU, CU), (CN, S)])
@pytest.mark.parametrize("R", [1, 2, 3, 8, 16, 17, 32, 64, 100, 128, 130])
def test_spmm(dims, nnz, seed, attr, R, tile_items):
    if tile_items == 37 and R not in (2, 17, 64):
        pytest.skip("odd tiling is sampled on a few widths")
    coords, val = synth.random_coo(dims, nnz, seed)
    c, v = _np(coords), val.numpy()
    B = synth.random_dense((dims[1], R), seed).numpy()
    want, norm = oracle.spmm(c, v, dims, B)
    A = upload_packed(oracle.pack(c, v, dims, (0, 1), attr))
    C = torch.full((dims[0], R), float("nan"), dtype=torch.float64, device="cuda")
    comet.spmm(A, dev(B), C)
    assert_close(C, want, norm, what=f"spmm R={R}")


def test_spmm_strided_and_unaligned_operands():
    dims, R = (120, 90), 16
    coords, val = synth.random_coo(dims, 1500, 3)
    c, v = _np(coords), val.numpy()
    B = synth.random_dense((dims[1], R), 3).numpy()
    want, norm = oracle.spmm(c, v, dims, B)
    A = upload_packed(oracle.pack(c, v, dims, (0, 1), (D, CU)))
    for ldb, ldc, off in [(R + 4, R + 2, 0), (R + 1, R + 3, 0), (R, R, 1)]:
        Bbuf = torch.zeros(dims[1] * ldb + 8, dtype=torch.float64, device="cuda")
        Bd = Bbuf[off:off + dims[1] * ldb].view(dims[1], ldb)[:, :R]
        Bd.copy_(dev(B))
        Cbuf = torch.full((dims[0] * ldc + 8,), 7.0, dtype=torch.float64, device="cuda")
        Cd = Cbuf[off:off + dims[0] * ldc].view(dims[0], ldc)[:, :R]
        comet.spmm(A, Bd, Cd)
        assert_close(Cd, want, norm, what=f"spmm ld=({ldb},{ldc}) off={off}")
        if ldc > R:
            assert bool((Cbuf[off:off + dims[0] * ldc].view(dims[0], ldc)[:, R:] == 7.0).all())   # padding untouched


def test_exact_on_small_integers():
    dims = (90, 70)
    coords, val = synth.random_coo(dims, 2500, 11, integer_values=True)
    c, v = _np(coords), val.numpy()
    B = synth.random_dense((dims[1], 32), 11, integer_values=True).numpy()
    want, _ = oracle.spmm(c, v, dims, B)
    A = upload_packed(oracle.pack(c, v, dims, (0, 1), (D, CU)))
    assert_equal_arrays(comet.spmm(A, dev(B)), want, "integer spmm")
    assert_equal_arrays(comet.spmv(A, dev(B[:, 0].copy())), want[:, 0], "integer spmv")


TENSOR_CASES = [((20, 18, 16), 900, 1), ((50, 40, 30), 6000, 2), ((1, 30, 30), 300, 3), ((30, 1, 30), 300, 4),
                ((30, 30, 1), 300, 5), ((12, 11, 10), 1320, 6), ((40, 40, 40), 1, 7), ((40, 40, 40), 0, 8),
                ((2000, 5, 7), 500, 9)]


@pytest.mark.parametrize("dims,nnz,seed", TENSOR_CASES)
@pytest.mark.parametrize("mode", [0, 1, 2])
def test_ttv_ttm(dims, nnz, seed, mode, tile_items, seg_dot_path):
    coords, val = synth.random_coo(dims, nnz, seed)
    c, v = _np(coords), val.numpy()
    kept = [m for m in range(3) if m != mode]
    mode_order = (kept[0], kept[1], mode)                       # contracted mode stored last
    pk = oracle.pack(c, v, dims, mode_order, (CU, CU, CU))
    X = upload_packed(pk)
    vec = synth.random_dense((dims[mode],), seed).numpy()
    keys, want, norm = oracle.ttv(c, v, dims, mode, vec)
    for out_attr in [(D, CU), (CU, CU)]:
        Y = comet.ttv_symbolic(X, mode, out_attr)
        Y.val.fill_(float("nan"))
        comet.ttv(X, mode, dev(vec), Y)
        assert_close(Y.val, want, norm, what="ttv")
        # structure: the sparse matrix over the kept modes, packed in the asked format
        ka, kb = keys // dims[kept[1]], keys % dims[kept[1]]
        ref = oracle.pack([ka, kb], np.ones(len(keys)), (dims[kept[0]], dims[kept[1]]), (0, 1), out_attr)
        for l in range(2):
            assert_equal_arrays(Y.pos(l), ref.pos[l], f"ttv pos{l}")
            assert_equal_arrays(Y.crd(l), ref.crd[l], f"ttv crd{l}")
    for R in (1, 4, 16, 5):
        U = synth.random_dense((dims[mode], R), seed + 1).numpy()
        _, wantm, normm = oracle.ttm(c, v, dims, mode, U)
        Z = comet.ttm_symbolic(X, mode, R)
        Z.val.fill_(float("nan"))
        comet.ttm(X, mode, dev(U), Z)
        assert_close(Z.val.reshape(-1, R), wantm, normm, what=f"ttm R={R}")
        for l in range(2):
            assert_equal_arrays(Z.pos(l), pk.pos[l], f"ttm pos{l}")
            assert_equal_arrays(Z.crd(l), pk.crd[l], f"ttm crd{l}")


@pytest.mark.parametrize("dims,nnz,seed", TENSOR_CASES)
@pytest.mark.parametrize("mode", [0, 1, 2])
def test_ttv_ttm_from_sorted_coo(dims, nnz, seed, mode, tile_items):
    """[CN,S,S] input: the fibers are derived from the sorted coordinates in the symbolic call; values and
    structure must equal those from the CSF tensor of the same entries."""
    coords, val = synth.random_coo(dims, nnz, seed)
    c, v = _np(coords), val.numpy()
    kept = [m for m in range(3) if m != mode]
    mode_order = (kept[0], kept[1], mode)
    X = upload_packed(oracle.pack(c, v, dims, mode_order, (CN, S, S)))
    csf = oracle.pack(c, v, dims, mode_order, (CU, CU, CU))
    vec = synth.random_dense((dims[mode],), seed).numpy()
    keys, want, norm = oracle.ttv(c, v, dims, mode, vec)
    for out_attr in [(D, CU), (CU, CU)]:
        Y = comet.ttv_symbolic(X, mode, out_attr)
        comet.validate(Y)
        Y.val.fill_(float("nan"))
        comet.ttv(X, mode, dev(vec), Y)
        assert_close(Y.val, want, norm, what="coo ttv")
        ka, kb = keys // dims[kept[1]], keys % dims[kept[1]]
        ref = oracle.pack([ka, kb], np.ones(len(keys)), (dims[kept[0]], dims[kept[1]]), (0, 1), out_attr)
        for l in range(2):
            assert_equal_arrays(Y.pos(l), ref.pos[l], f"coo ttv pos{l}")
            assert_equal_arrays(Y.crd(l), ref.crd[l], f"coo ttv crd{l}")
        comet.ttv(X, mode, dev(vec), Y)                                  # the numeric phase can be repeated
        assert_close(Y.val, want, norm, what="coo ttv again")
    for R in (1, 16, 5):
        U = synth.random_dense((dims[mode], R), seed + 1).numpy()
        _, wantm, normm = oracle.ttm(c, v, dims, mode, U)
        Z = comet.ttm_symbolic(X, mode, R)
        Z.val.fill_(float("nan"))
        comet.ttm(X, mode, dev(U), Z)
        assert_close(Z.val.reshape(-1, R), wantm, normm, what=f"coo ttm R={R}")
        assert Z.attr == (CU, CU, D)
        for l in range(2):
            assert_equal_arrays(Z.pos(l), csf.pos[l], f"coo ttm pos{l}")
            assert_equal_arrays(Z.crd(l), csf.crd[l], f"coo ttm crd{l}")
        assert Z.pos(2).tolist() == [R]


ORDER4_CASES = [((9, 8, 7, 6), 900, 1), ((20, 15, 12, 10), 6000, 2), ((1, 12, 12, 12), 300, 3),
                ((12, 12, 12, 1), 300, 4), ((6, 5, 4, 3), 360, 5), ((10, 10, 10, 10), 0, 6), ((400, 3, 5, 4), 500, 7)]


@pytest.mark.parametrize("dims,nnz,seed", ORDER4_CASES)
@pytest.mark.parametrize("mode", [0, 1, 2, 3])
def test_ttv_ttm_order4_csf(dims, nnz, seed, mode, tile_items):
    """4-order tensors in CSF [CU,CU,CU,CU], contracted mode stored last: the result's structure is X's three
    upper levels, values against the order-N oracle."""
    coords, val = synth.random_coo(dims, nnz, seed)
    c, v = _np(coords), val.numpy()
    kept = [m for m in range(4) if m != mode]
    mode_order = (kept[0], kept[1], kept[2], mode)
    pk = oracle.pack(c, v, dims, mode_order, (CU, CU, CU, CU))
    X = upload_packed(pk)
    vec = synth.random_dense((dims[mode],), seed).numpy()
    keys, want, norm = oracle.ttm_n(c, v, dims, mode, vec)
    Y = comet.ttv_symbolic(X, mode)
    comet.validate(Y)
    assert Y.attr == (CU, CU, CU) and Y.dims == tuple(dims[m] for m in kept) and Y.c.nnz == len(keys)
    Y.val.fill_(float("nan"))
    comet.ttv(X, mode, dev(vec), Y)
    assert_close(Y.val, want[:, 0], norm[:, 0], what="ttv order 4")
    for l in range(3):
        assert_equal_arrays(Y.pos(l), pk.pos[l], f"ttv4 pos{l}")
        assert_equal_arrays(Y.crd(l), pk.crd[l], f"ttv4 crd{l}")
    # the leaf coordinates of Y enumerate the kept-coordinate keys in ascending order
    for R in (1, 16, 5):
        U = synth.random_dense((dims[mode], R), seed + 1).numpy()
        _, wantm, normm = oracle.ttm_n(c, v, dims, mode, U)
        Z = comet.ttm_symbolic(X, mode, R)
        assert Z.attr == (CU, CU, CU, D) and Z.pos(3).tolist() == [R]
        assert Z.dims == tuple(R if m == mode else d for m, d in enumerate(dims))
        Z.val.fill_(float("nan"))
        comet.ttm(X, mode, dev(U), Z)
        assert_close(Z.val.reshape(-1, R), wantm, normm, what=f"ttm order 4 R={R}")
        for l in range(3):
            assert_equal_arrays(Z.pos(l), pk.pos[l], f"ttm4 pos{l}")
            assert_equal_arrays(Z.crd(l), pk.crd[l], f"ttm4 crd{l}")


@pytest.mark.parametrize("dims,nnz,seed", ORDER4_CASES)
@pytest.mark.parametrize("mode", [0, 3])
def test_ttv_ttm_order4_from_sorted_coo(dims, nnz, seed, mode):
    """4-order tensors in sorted COO [CN,S,S,S], contracted mode stored last: the symbolic call derives the three
    upper CSF levels (bit-exact against the oracle's CSF packing), the values against the order-N oracle."""
    coords, val = synth.random_coo(dims, nnz, seed)
    c, v = _np(coords), val.numpy()
    kept = [m for m in range(4) if m != mode]
    mode_order = (kept[2], kept[0], kept[1], mode)
    X = upload_packed(oracle.pack(c, v, dims, mode_order, (CN, S, S, S)))
    csf = oracle.pack(c, v, dims, mode_order, (CU, CU, CU, CU))
    # the oracle lists fibers by increasing MODE; the storage lists them in (kept[2], kept[0], kept[1]) order
    keys, want, norm = oracle.ttm_n(c, v, dims, mode, synth.random_dense((dims[mode],), seed).numpy())
    k0 = keys // (dims[kept[1]] * dims[kept[2]])
    k1 = (keys // dims[kept[2]]) % dims[kept[1]]
    k2 = keys % dims[kept[2]]
    stored = np.lexsort((k1, k0, k2)) if len(keys) else np.zeros(0, dtype=np.int64)
    vec = synth.random_dense((dims[mode],), seed).numpy()
    Y = comet.ttv_symbolic(X, mode)
    assert Y.attr == (CU, CU, CU) and Y.c.nnz == len(keys)
    for l in range(3):
        assert_equal_arrays(Y.pos(l), csf.pos[l], f"coo4 ttv pos{l}")
        assert_equal_arrays(Y.crd(l), csf.crd[l], f"coo4 ttv crd{l}")
    Y.val.fill_(float("nan"))
    comet.ttv(X, mode, dev(vec), Y)
    assert_close(Y.val, want[stored, 0], norm[stored, 0], what="ttv order 4 from coo")
    for R in (1, 16, 5):
        U = synth.random_dense((dims[mode], R), seed + 1).numpy()
        _, wantm, normm = oracle.ttm_n(c, v, dims, mode, U)
        Z = comet.ttm_symbolic(X, mode, R)
        assert Z.attr == (CU, CU, CU, D) and Z.pos(3).tolist() == [R]
        Z.val.fill_(float("nan"))
        comet.ttm(X, mode, dev(U), Z)
        assert_close(Z.val.reshape(-1, R), wantm[stored], normm[stored], what=f"ttm order 4 from coo R={R}")
        for l in range(3):
            assert_equal_arrays(Z.pos(l), csf.pos[l], f"coo4 ttm pos{l}")
            assert_equal_arrays(Z.crd(l), csf.crd[l], f"coo4 ttm crd{l}")


@pytest.mark.parametrize("dims,nnz,seed", ORDER4_CASES)
@pytest.mark.parametrize("mode_order", [(0, 1, 2, 3), (3, 1, 0, 2)])
@pytest.mark.parametrize("attr", [(CN, S, S, S), (CU, CU, CU, CU)])
def test_mttkrp_order4_every_mode(dims, nnz, seed, mode_order, attr):
    coords, val = synth.random_coo(dims, nnz, seed)
    c, v = _np(coords), val.numpy()
    X = upload_packed(oracle.pack(c, v, dims, mode_order, attr))
    for R in (1, 5, 16, 40):
        F = [synth.random_dense((d, R), seed, 60 + m).numpy() for m, d in enumerate(dims)]
        for mode in range(4):
            want, norm = oracle.mttkrp_n(c, v, dims, mode, F)
            out = torch.full((dims[mode], R), float("nan"), dtype=torch.float64, device="cuda")
            comet.mttkrp(X, mode, [None if m == mode else dev(f) for m, f in enumerate(F)], out)
            assert_close(out, want, norm, what=f"mttkrp4 mode {mode} of {mode_order} {attr} R={R}")


def test_mttkrp_order4_integers_exact_and_fp32():
    dims = (12, 10, 9, 8)
    coords, val = synth.random_coo(dims, 3000, 4, integer_values=True)
    c, v = _np(coords), val.numpy()
    F = [synth.random_dense((d, 6), 4, 60 + m, integer_values=True).numpy() for m, d in enumerate(dims)]
    for attr in [(CN, S, S, S), (CU, CU, CU, CU)]:
        pk = oracle.pack(c, v, dims, (1, 0, 3, 2), attr)
        X = upload_packed(pk)
        pos = [dev(p, torch.int32) if p.size else None for p in pk.pos]
        crd = [dev(x, torch.int32) if x.size else None for x in pk.crd]
        X32 = comet.SpTensor.from_arrays(pk.dims, pk.mode_order, pk.attr, pos, crd, dev(pk.val.astype(np.float32)))
        for mode in range(4):
            want, _ = oracle.mttkrp_n(c, v, dims, mode, F)
            got = comet.mttkrp(X, mode, [None if m == mode else dev(f) for m, f in enumerate(F)])
            assert_equal_arrays(got, want, "integer mttkrp4")
            got32 = comet.mttkrp(X32, mode, [None if m == mode else dev(f.astype(np.float32)) for m, f in enumerate(F)])
            assert got32.dtype == torch.float32 and np.array_equal(got32.cpu().numpy().astype(np.float64), want)


def test_order4_packed_on_the_device_then_contracted():
    dims = (30, 25, 20, 15)
    coords, val = synth.random_coo(dims, 20000, 9)
    c, v = _np(coords), val.numpy()
    X = comet.pack([t.cuda() for t in coords], val.cuda(), dims, (3, 1, 0, 2), (CU, CU, CU, CU))
    vec = synth.random_dense((dims[2],), 9).numpy()
    keys, want, norm = oracle.ttm_n(c, v, dims, 2, vec)
    # oracle keys are in increasing MODE order (0,1,3); the stored order is (3,1,0): bring the oracle's fibers into
    # the stored order and compare fiber by fiber with each fiber's own normaliser
    k0, k1, k3 = keys // (dims[1] * dims[3]), (keys // dims[3]) % dims[1], keys % dims[3]
    stored = np.lexsort((k0, k1, k3))
    Y = comet.ttv(X, 2, dev(vec))
    assert Y.c.nnz == len(want)
    assert_close(Y.val, want[stored, 0], norm[stored, 0], what="ttv of a device-packed 4-order tensor")


@pytest.mark.parametrize("dims,nnz,seed", TENSOR_CASES)
@pytest.mark.parametrize("attr", [(CU, CU, CU), (CN, S, S)])
def test_ttm_mode_generic_output(dims, nnz, seed, attr):
    """[CN,S,D] result: one coordinate pair per stored fiber, the same values as the default [CU,CU,D] result."""
    coords, val = synth.random_coo(dims, nnz, seed)
    c, v = _np(coords), val.numpy()
    mode, R = 2, 6
    X = upload_packed(oracle.pack(c, v, dims, (0, 1, 2), attr))
    U = synth.random_dense((dims[mode], R), seed + 1).numpy()
    keys, want, norm = oracle.ttm(c, v, dims, mode, U)
    Z = comet.ttm_symbolic(X, mode, R, (CN, S, D))
    assert Z.attr == (CN, S, D) and Z.dims == (dims[0], dims[1], R) and Z.c.nnz == len(keys) * R
    assert Z.pos(0).tolist() == [0, len(keys)] and Z.pos(2).tolist() == [R]
    assert_equal_arrays(Z.crd(0), (keys // dims[1]).astype(np.int32), "fiber coordinates of mode 0")
    assert_equal_arrays(Z.crd(1), (keys % dims[1]).astype(np.int32), "fiber coordinates of mode 1")
    Z.val.fill_(float("nan"))
    comet.ttm(X, mode, dev(U), Z)
    assert_close(Z.val.reshape(-1, R), want, norm, what="mode-generic ttm")
    with pytest.raises(comet.CometError) as e:
        comet.ttm_symbolic(X, mode, R, (D, CU, D))
    assert e.value.status == -2


def test_ttv_numeric_phase_rejects_a_result_built_for_another_tensor():
    dims = (12, 11, 10)
    coords, val = synth.random_coo(dims, 400, 3)
    c, v = _np(coords), val.numpy()
    Xcoo = upload_packed(oracle.pack(c, v, dims, (0, 1, 2), (CN, S, S)))
    Xcsf = upload_packed(oracle.pack(c, v, dims, (0, 1, 2), (CU, CU, CU)))
    Y = comet.ttv_symbolic(Xcsf, 2)            # carries no fiber boundaries: a COO numeric call cannot use it
    with pytest.raises(comet.CometError) as e:
        comet.ttv(Xcoo, 2, dev(np.ones(10)), Y)
    assert e.value.status == -1


@pytest.mark.parametrize("dims,nnz,seed", TENSOR_CASES)
@pytest.mark.parametrize("mode", [0, 1, 2])
@pytest.mark.parametrize("attr", [(CN, S, S), (CU, CU, CU)])
def test_mttkrp(dims, nnz, seed, mode, attr, tile_items):
    coords, val = synth.random_coo(dims, nnz, seed)
    c, v = _np(coords), val.numpy()
    kept = [m for m in range(3) if m != mode]
    mode_order = (mode, kept[0], kept[1])                       # output mode stored first
    X = upload_packed(oracle.pack(c, v, dims, mode_order, attr))
    for R in (1, 8, 32, 7):
        F = [synth.random_dense((d, R), seed, 60 + m).numpy() for m, d in enumerate(dims)]
        want, norm = oracle.mttkrp(c, v, dims, mode, F)
        out = torch.full((dims[mode], R), float("nan"), dtype=torch.float64, device="cuda")
        comet.mttkrp(X, mode, [None if m == mode else dev(f) for m, f in enumerate(F)], out)
        assert_close(out, want, norm, what=f"mttkrp R={R}")


@pytest.mark.parametrize("dims,nnz,seed", TENSOR_CASES)
@pytest.mark.parametrize("mode_order", [(0, 1, 2), (2, 0, 1), (1, 2, 0)])
@pytest.mark.parametrize("attr", [(CN, S, S), (CU, CU, CU)])
def test_mttkrp_every_mode_of_a_fixed_tensor(dims, nnz, seed, mode_order, attr):
    """All three modes on ONE packed tensor (the all-modes sequence of CP-ALS): the mode stored first takes
    the deterministic kernels, the other two accumulate with atomic adds on the tensor as stored."""
    coords, val = synth.random_coo(dims, nnz, seed)
    c, v = _np(coords), val.numpy()
    X = upload_packed(oracle.pack(c, v, dims, mode_order, attr))
    for R in (1, 3, 16, 40):
        F = [synth.random_dense((d, R), seed, 60 + m).numpy() for m, d in enumerate(dims)]
        for mode in range(3):
            want, norm = oracle.mttkrp(c, v, dims, mode, F)
            out = torch.full((dims[mode], R), float("nan"), dtype=torch.float64, device="cuda")
            comet.mttkrp(X, mode, [None if m == mode else dev(f) for m, f in enumerate(F)], out)
            assert_close(out, want, norm, what=f"mttkrp mode {mode} of {mode_order} R={R}")


def _skewed_leaf_coo(dims, nnz, seed):
    """Distinct cells whose last coordinate is drawn with very unequal frequencies (a few popular values)."""
    g = np.random.default_rng(seed)
    i = g.integers(0, dims[0], 3 * nnz)
    j = g.integers(0, dims[1], 3 * nnz)
    k = np.minimum((dims[2] * g.random(3 * nnz) ** 4).astype(np.int64), dims[2] - 1)
    cells = np.unique((i * dims[1] + j) * dims[2] + k)
    cells = g.permutation(cells)[:nnz]
    c = [(cells // (dims[1] * dims[2])).astype(np.int32), (cells // dims[2] % dims[1]).astype(np.int32),
         (cells % dims[2]).astype(np.int32)]
    return c, g.uniform(-1.0, 1.0, cells.size)


@pytest.mark.parametrize("dims,nnz", [((40, 30, 500), 20000), ((7, 9, 20), 700), ((300, 200, 3000), 60000)])
@pytest.mark.parametrize("dtype", ["f64", "f32"])
@pytest.mark.parametrize("attr,modes", [((CU, CU, CU), (2,)), ((CN, S, S), (1, 2))])
def test_mttkrp_with_popular_rows_in_shared_memory(dims, nnz, dtype, attr, modes, monkeypatch):
    """The per-entry kernel that keeps the most popular output rows in shared memory (CSF: leaf mode; COO: both
    non-root modes), forced on small tensors (by default only large ones take it): fewer rows than slots, more
    rows than slots, R below, at and above a warp's width, entries that straddle the 32-fiber window."""
    monkeypatch.setenv("COMET_MTTKRP_HOT_ROWS", "1")
    c, v = _skewed_leaf_coo(dims, nnz, 11)
    if dtype == "f32":
        v = v.astype(np.float32).astype(np.float64)
    pk = oracle.pack(c, v, dims, (0, 1, 2), attr)
    if dtype == "f32":
        pos = [dev(p, torch.int32) if p.size else None for p in pk.pos]
        crd = [dev(q, torch.int32) if q.size else None for q in pk.crd]
        X = comet.SpTensor.from_arrays(pk.dims, pk.mode_order, pk.attr, pos, crd, dev(pk.val.astype(np.float32)))
    else:
        X = upload_packed(pk)
    tdt = torch.float32 if dtype == "f32" else torch.float64
    for R in (1, 5, 32, 40, 64):
        F = [synth.random_dense((d, R), 11, 60 + m).numpy() for m, d in enumerate(dims)]
        if dtype == "f32":
            F = [f.astype(np.float32).astype(np.float64) for f in F]
        for mode in modes:
            want, norm = oracle.mttkrp(c, v, dims, mode, F)
            out = torch.full((dims[mode], R), float("nan"), dtype=tdt, device="cuda")
            comet.mttkrp(X, mode, [None if m == mode else dev(f).to(tdt) for m, f in enumerate(F)], out)
            assert_close(out.double(), want, norm, tol=FP64_TOL if dtype == "f64" else 4e-7,
                         what=f"mttkrp {attr} mode {mode} {dtype} R={R}")
    if dtype == "f64":                                   # the general kernel on the same input
        monkeypatch.setenv("COMET_MTTKRP_HOT_ROWS", "0")
        F = [synth.random_dense((d, 5), 11, 60 + m).numpy() for m, d in enumerate(dims)]
        for mode in modes:
            want, norm = oracle.mttkrp(c, v, dims, mode, F)
            out0 = torch.full((dims[mode], 5), float("nan"), dtype=torch.float64, device="cuda")
            comet.mttkrp(X, mode, [None if m == mode else dev(f) for m, f in enumerate(F)], out0)
            assert_close(out0, want, norm, what=f"mttkrp {attr} mode {mode}, general kernel")


def test_mttkrp_non_root_strided_output_and_integers():
    dims = (25, 20, 15)
    coords, val = synth.random_coo(dims, 2000, 5, integer_values=True)
    c, v = _np(coords), val.numpy()
    R = 6
    F = [synth.random_dense((d, R), 5, 60 + m, integer_values=True).numpy() for m, d in enumerate(dims)]
    for attr in [(CN, S, S), (CU, CU, CU)]:
        X = upload_packed(oracle.pack(c, v, dims, (0, 1, 2), attr))
        for mode in (1, 2):
            want, _ = oracle.mttkrp(c, v, dims, mode, F)
            buf = torch.full((dims[mode], R + 3), 7.0, dtype=torch.float64, device="cuda")
            comet.mttkrp(X, mode, [None if m == mode else dev(f) for m, f in enumerate(F)], buf[:, :R])
            assert_equal_arrays(buf[:, :R].contiguous(), want, "integer non-root mttkrp")   # exact sums: any order
            assert bool((buf[:, R:] == 7.0).all())                                          # padding untouched


def test_mttkrp_exact_on_small_integers():
    dims = (25, 20, 15)
    coords, val = synth.random_coo(dims, 2000, 5, integer_values=True)
    c, v = _np(coords), val.numpy()
    F = [synth.random_dense((d, 16), 5, 60 + m, integer_values=True).numpy() for m, d in enumerate(dims)]
    want, _ = oracle.mttkrp(c, v, dims, 0, F)
    for attr in [(CN, S, S), (CU, CU, CU)]:
        X = upload_packed(oracle.pack(c, v, dims, (0, 1, 2), attr))
        assert_equal_arrays(comet.mttkrp(X, 0, [None, dev(F[1]), dev(F[2])]), want, "integer mttkrp")


def test_spmm_from_host_buffers():
    """The end-to-end call the benchmark times: pinned host COO + B in, C out."""
    case = synth.make(2, scale=1 / 512)
    c, v = _np(case.coords), case.val.numpy()
    want, norm = oracle.spmm(c, v, case.dims, case.dense["B"].numpy())
    h_coords = [t.pin_memory() for t in case.coords]
    h_val, h_B = case.val.pin_memory(), case.dense["B"].pin_memory()
    h_C = torch.full((case.dims[0], case.R), float("nan"), dtype=torch.float64).pin_memory()
    for _ in range(2):                                  # the second call reuses the copy streams
        h_C.fill_(float("nan"))
        comet.spmm_from_host(h_coords, h_val, case.dims, h_B, h_C)
        assert_close(h_C, want, norm, what="spmm_from_host")


@pytest.mark.parametrize("R,chunk_bytes", [(64, None), (40, None), (5, None), (64, "128"), (64, "0"), (33, "64")])
@pytest.mark.parametrize("dtype", ["f64", "f32"])
def test_spmm_from_host_column_chunks(R, chunk_bytes, dtype, monkeypatch):
    """comet_spmm_from_host with B and C cut into column chunks: even and ragged chunk counts, one chunk, strided
    host matrices (leading dimension above R, padding untouched), pageable as well as pinned memory, an empty
    matrix, and a bad coordinate reported as a status."""
    if chunk_bytes is None:
        monkeypatch.delenv("COMET_HOST_CHUNK_BYTES", raising=False)
    else:
        monkeypatch.setenv("COMET_HOST_CHUNK_BYTES", chunk_bytes)
    tdt = torch.float32 if dtype == "f32" else torch.float64
    dims = (300, 200)
    coords, val = synth.random_coo(dims, 4000, 21)
    Bm = synth.random_dense((dims[1], R), 21, 3)
    if dtype == "f32":
        val, Bm = val.float().double(), Bm.float().double()
    want, norm = oracle.spmm(_np(coords), val.numpy(), dims, Bm.numpy())
    tol = FP64_TOL if dtype == "f64" else 4e-7
    h_coords = [t.pin_memory() for t in coords]
    h_val = val.to(tdt).pin_memory()
    h_Bbuf = torch.full((dims[1], R + 3), 5.0, dtype=tdt).pin_memory()
    h_Bbuf[:, :R] = Bm.to(tdt)
    h_Cbuf = torch.full((dims[0], R + 2), 7.0, dtype=tdt).pin_memory()
    comet.spmm_from_host(h_coords, h_val, dims, h_Bbuf[:, :R], h_Cbuf[:, :R])
    assert_close(h_Cbuf[:, :R].double(), want, norm, tol=tol, what=f"spmm_from_host R={R} chunks of {chunk_bytes}")
    assert bool((h_Cbuf[:, R:] == 7.0).all())
    # pageable host memory: correct, only slower
    p_C = torch.full((dims[0], R), float("nan"), dtype=tdt)
    comet.spmm_from_host([t.clone() for t in coords], val.to(tdt), dims, Bm.to(tdt).contiguous(), p_C)
    assert_close(p_C.double(), want, norm, tol=tol, what="spmm_from_host, pageable memory")
    # no entries: C = 0
    e_C = torch.full((dims[0], R), float("nan"), dtype=tdt).pin_memory()
    empty = [torch.zeros(0, dtype=torch.int32).pin_memory() for _ in range(2)]
    comet.spmm_from_host(empty, torch.zeros(0, dtype=tdt).pin_memory(), dims, h_Bbuf[:, :R], e_C)
    assert bool((e_C == 0).all())
    # a coordinate outside the matrix is a status, and the handle keeps working
    bad = [h_coords[0].clone(), h_coords[1].clone()]
    bad[1][7] = dims[1]
    with pytest.raises(comet.CometError) as err:
        comet.spmm_from_host(bad, h_val, dims, h_Bbuf[:, :R], h_Cbuf[:, :R])
    assert err.value.status == -3
    comet.spmm_from_host(h_coords, h_val, dims, h_Bbuf[:, :R], h_Cbuf[:, :R])
    assert_close(h_Cbuf[:, :R].double(), want, norm, tol=tol, what="spmm_from_host after an error")


def test_results_are_reproducible_run_to_run():
    case = synth.make(2, scale=1 / 256)
    c, v = _np(case.coords), case.val.numpy()
    A = upload_packed(oracle.pack(c, v, case.dims, (0, 1), (D, CU)))
    B = case.dense["B"].cuda()
    first = comet.spmm(A, B).clone()
    for _ in range(3):
        assert torch.equal(comet.spmm(A, B), first)


@pytest.mark.parametrize("config", [1, 2, 3, 4, 5])
def test_scaled_workloads(config, seg_dot_path):
    """The five benchmark workloads at 1/64 scale (several tiles, ragged tails, skewed segments)."""
    case = synth.make(config, scale=1 / 64)
    c, v = _np(case.coords), case.val.numpy()
    if config == 1:
        want, norm = oracle.spmv(c, v, case.dims, case.dense["x"].numpy())
        A = upload_packed(oracle.pack(c, v, case.dims, (0, 1), (D, CU)))
        assert_close(comet.spmv(A, case.dense["x"].cuda()), want, norm, what="C1")
    elif config == 2:
        want, norm = oracle.spmm(c, v, case.dims, case.dense["B"].numpy())
        A = upload_packed(oracle.pack(c, v, case.dims, (0, 1), (D, CU)))
        assert_close(comet.spmm(A, case.dense["B"].cuda()), want, norm, what="C2")
    elif config == 3:
        _, want, norm = oracle.ttv(c, v, case.dims, 2, case.dense["v"].numpy())
        X = upload_packed(oracle.pack(c, v, case.dims, (0, 1, 2), (CU, CU, CU)))
        assert_close(comet.ttv(X, 2, case.dense["v"].cuda()).val, want, norm, what="C3")
    elif config == 4:
        _, want, norm = oracle.ttm(c, v, case.dims, 2, case.dense["U"].numpy())
        X = upload_packed(oracle.pack(c, v, case.dims, (0, 1, 2), (CU, CU, CU)))
        assert_close(comet.ttm(X, 2, case.dense["U"].cuda()).val.reshape(-1, case.R), want, norm, what="C4")
    else:
        F = [None, case.dense["B"].numpy(), case.dense["C"].numpy()]
        want, norm = oracle.mttkrp(c, v, case.dims, 0, F)
        Fd = [None, case.dense["B"].cuda(), case.dense["C"].cuda()]
        for attr in [(CN, S, S), (CU, CU, CU)]:
            X = upload_packed(oracle.pack(c, v, case.dims, (0, 1, 2), attr))
            assert_close(comet.mttkrp(X, 0, Fd), want, norm, what=f"C5 {attr}")


def test_argument_errors_are_reported_not_raised_by_cuda():
    A = upload_packed(oracle.pack([[0], [1]], [1.0], (2, 2), (0, 1), (D, CU)))
    B = torch.ones((2, 4), dtype=torch.float64, device="cuda")
    with pytest.raises(comet.CometError) as e:
        comet.spmm(A, B, torch.empty((2, 2), dtype=torch.float64, device="cuda"))     # ldc < R
    assert e.value.status == -1
    X = upload_packed(oracle.pack([[0], [1], [1]], [1.0], (2, 2, 2), (0, 1, 2), (CU, CU, CU)))
    with pytest.raises(comet.CometError) as e:
        comet.ttv(X, 0, torch.ones(2, dtype=torch.float64, device="cuda"))             # mode 0 is not stored last
    assert e.value.status == -2
    with pytest.raises(comet.CometError) as e:
        comet.mttkrp(X, 3, [B[:, :1], B[:, :1], None])                                 # no such mode
    assert e.value.status == -1
    Xd = upload_packed(oracle.pack([[0], [1], [1]], [1.0], (2, 2, 2), (0, 1, 2), (D, CU, CU)))
    with pytest.raises(comet.CometError) as e:
        comet.mttkrp(Xd, 0, [None, B[:, :1], B[:, :1]])                                # MTTKRP takes COO or CSF
    assert e.value.status == -2
