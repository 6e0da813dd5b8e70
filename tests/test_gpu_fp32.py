"""GPU parity of the fp32 value type: values, dense operands and outputs are float32, the kernels
multiply and accumulate in double and round once on the store. The oracle gets the SAME float32 values
(widened to double, which is exact), so the only differences are the final rounding to float32 and,
on a row that spans several tiles, one more rounding when its carry is added.

Bound asserted: 1e-5 * sum|terms| (the stated fp32 tolerance) and, tighter, 3 float32 roundings."""
import numpy as np
import pytest
import torch

import oracle
import synth
from oracle import D, CU, CN, S

pytestmark = pytest.mark.gpu

comet = pytest.importorskip("paper_2102_05187_b200")
from gpu_util import assert_close, assert_equal_arrays, dev  # noqa: E402

FP32_TOL = 1e-5                      # the tolerance stated for fp32 results
FP32_TIGHT = 3 * 2.0 ** -24          # what double accumulation actually leaves: the store and carry roundings


@pytest.fixture(autouse=True)
def _need_gpu(cuda_device):
    yield


@pytest.fixture(params=[None, 8, 37])
def tile_items(request, monkeypatch):
    if request.param is None:
        monkeypatch.delenv("COMET_TILE_ITEMS", raising=False)
    else:
        monkeypatch.setenv("COMET_TILE_ITEMS", str(request.param))
    return request.param


@pytest.fixture(params=["default", "resident", "stream", "stream-short-spans", "stream2", "stream2-short-spans"])
def seg_dot_path(request, monkeypatch):
    monkeypatch.delenv("COMET_SEG_DOT_KERNEL", raising=False)
    monkeypatch.delenv("COMET_STREAM_SPAN", raising=False)
    if request.param == "resident":
        monkeypatch.setenv("COMET_SEG_DOT_KERNEL", "resident")
    elif request.param.startswith("stream"):
        monkeypatch.setenv("COMET_SEG_DOT_KERNEL", "stream2" if request.param.startswith("stream2") else "stream")
        if request.param.endswith("short-spans"):
            monkeypatch.setenv("COMET_STREAM_SPAN", "128")
    return request.param


def f32(a):
    """Round to float32 and widen again: what the oracle is fed, exactly what the device holds."""
    return np.asarray(a, dtype=np.float32).astype(np.float64)


def dev32(a):
    return dev(np.asarray(a, dtype=np.float32))


def upload32(pk):
    pos = [dev(p, torch.int32) if p.size else None for p in pk.pos]
    crd = [dev(c, torch.int32) if c.size else None for c in pk.crd]
    return comet.SpTensor.from_arrays(pk.dims, pk.mode_order, pk.attr, pos, crd, dev32(pk.val))


def check(got, want, norm, what):
    assert got.dtype == torch.float32, what
    got = got.double()
    assert_close(got, want, norm, tol=FP32_TOL, what=what)
    assert_close(got, want, norm, tol=FP32_TIGHT, what=what + " (tight)")


def _coo(dims, nnz, seed):
    coords, val = synth.random_coo(dims, nnz, seed)
    return [c.numpy() for c in coords], f32(val.numpy())


MATRIX_CASES = [((64, 48), 700, 1), ((300, 200), 5000, 2), ((1, 500), 300, 3), ((500, 1), 200, 4),
                ((40, 40), 1600, 5), ((200, 300), 1, 6), ((200, 300), 0, 7), ((3000, 100), 400, 8)]


@pytest.mark.parametrize("dims,nnz,seed", MATRIX_CASES)
@pytest.mark.parametrize("attr", [(D, CU), (CU, CU), (CN, S)])
def test_spmv_fp32(dims, nnz, seed, attr, tile_items, seg_dot_path):
    c, v = _coo(dims, nnz, seed)
    x = f32(synth.random_dense((dims[1],), seed).numpy())
    want, norm = oracle.spmv(c, v, dims, x)
    A = upload32(oracle.pack(c, v, dims, (0, 1), attr))
    y = torch.full((dims[0],), float("nan"), dtype=torch.float32, device="cuda")
    comet.spmv(A, dev32(x), y)
    check(y, want, norm, "spmv fp32")


@pytest.mark.parametrize("dims,nnz,seed", MATRIX_CASES)
@pytest.mark.parametrize("attr", [(D, CU), (CU, CU), (CN, S)])
@pytest.mark.parametrize("R", [1, 3, 4, 8, 16, 17, 32, 64, 100, 128, 132, 260])
def test_spmm_fp32(dims, nnz, seed, attr, R, tile_items):
    if tile_items == 37 and R not in (4, 17, 64):
        pytest.skip("odd tiling is sampled on a few widths")
    c, v = _coo(dims, nnz, seed)
    B = f32(synth.random_dense((dims[1], R), seed).numpy())
    want, norm = oracle.spmm(c, v, dims, B)
    A = upload32(oracle.pack(c, v, dims, (0, 1), attr))
    C = torch.full((dims[0], R), float("nan"), dtype=torch.float32, device="cuda")
    comet.spmm(A, dev32(B), C)
    check(C, want, norm, f"spmm fp32 R={R}")


def test_spmm_fp32_strided_and_unaligned_operands():
    dims, R = (120, 90), 16
    c, v = _coo(dims, 1500, 3)
    B = f32(synth.random_dense((dims[1], R), 3).numpy())
    want, norm = oracle.spmm(c, v, dims, B)
    A = upload32(oracle.pack(c, v, dims, (0, 1), (D, CU)))
    for ldb, ldc, off in [(R + 4, R + 8, 0), (R + 1, R + 3, 0), (R, R, 1), (R, R, 2), (R + 2, R + 2, 3)]:
        Bbuf = torch.zeros(dims[1] * ldb + 8, dtype=torch.float32, device="cuda")
        Bd = Bbuf[off:off + dims[1] * ldb].view(dims[1], ldb)[:, :R]
        Bd.copy_(dev32(B))
        Cbuf = torch.full((dims[0] * ldc + 8,), 7.0, dtype=torch.float32, device="cuda")
        Cd = Cbuf[off:off + dims[0] * ldc].view(dims[0], ldc)[:, :R]
        comet.spmm(A, Bd, Cd)
        check(Cd, want, norm, f"spmm fp32 ld=({ldb},{ldc}) off={off}")
        if ldc > R:
            assert bool((Cbuf[off:off + dims[0] * ldc].view(dims[0], ldc)[:, R:] == 7.0).all())


def test_fp32_exact_on_small_integers():
    dims = (90, 70)
    coords, val = synth.random_coo(dims, 2500, 11, integer_values=True)
    c, v = [x.numpy() for x in coords], val.numpy()
    B = synth.random_dense((dims[1], 32), 11, integer_values=True).numpy()
    want, _ = oracle.spmm(c, v, dims, B)
    A = upload32(oracle.pack(c, v, dims, (0, 1), (D, CU)))
    assert np.array_equal(comet.spmm(A, dev32(B)).cpu().numpy().astype(np.float64), want)
    assert np.array_equal(comet.spmv(A, dev32(B[:, 0].copy())).cpu().numpy().astype(np.float64), want[:, 0])


TENSOR_CASES = [((20, 18, 16), 900, 1), ((50, 40, 30), 6000, 2), ((1, 30, 30), 300, 3), ((30, 30, 1), 300, 5),
                ((12, 11, 10), 1320, 6), ((40, 40, 40), 0, 8), ((2000, 5, 7), 500, 9)]


@pytest.mark.parametrize("dims,nnz,seed", TENSOR_CASES)
@pytest.mark.parametrize("mode", [0, 1, 2])
def test_ttv_ttm_fp32(dims, nnz, seed, mode, tile_items, seg_dot_path):
    c, v = _coo(dims, nnz, seed)
    kept = [m for m in range(3) if m != mode]
    pk = oracle.pack(c, v, dims, (kept[0], kept[1], mode), (CU, CU, CU))
    X = upload32(pk)
    vec = f32(synth.random_dense((dims[mode],), seed).numpy())
    _, want, norm = oracle.ttv(c, v, dims, mode, vec)
    for out_attr in [(D, CU), (CU, CU)]:
        Y = comet.ttv_symbolic(X, mode, out_attr)
        Y.val.fill_(float("nan"))
        comet.ttv(X, mode, dev32(vec), Y)
        check(Y.val, want, norm, "ttv fp32")
    for R in (1, 4, 16, 5, 64):
        U = f32(synth.random_dense((dims[mode], R), seed + 1).numpy())
        _, wantm, normm = oracle.ttm(c, v, dims, mode, U)
        Z = comet.ttm_symbolic(X, mode, R)
        Z.val.fill_(float("nan"))
        comet.ttm(X, mode, dev32(U), Z)
        check(Z.val.reshape(-1, R), wantm, normm, f"ttm fp32 R={R}")
        for l in range(2):
            assert_equal_arrays(Z.pos(l), pk.pos[l], f"ttm pos{l}")
            assert_equal_arrays(Z.crd(l), pk.crd[l], f"ttm crd{l}")


@pytest.mark.parametrize("dims,nnz,seed", TENSOR_CASES)
@pytest.mark.parametrize("mode", [0, 1, 2])
@pytest.mark.parametrize("attr", [(CN, S, S), (CU, CU, CU)])
def test_mttkrp_fp32(dims, nnz, seed, mode, attr, tile_items):
    c, v = _coo(dims, nnz, seed)
    kept = [m for m in range(3) if m != mode]
    X = upload32(oracle.pack(c, v, dims, (mode, kept[0], kept[1]), attr))
    for R in (1, 4, 8, 32, 7, 64, 130):
        F = [f32(synth.random_dense((d, R), seed, 60 + m).numpy()) for m, d in enumerate(dims)]
        want, norm = oracle.mttkrp(c, v, dims, mode, F)
        out = torch.full((dims[mode], R), float("nan"), dtype=torch.float32, device="cuda")
        comet.mttkrp(X, mode, [None if m == mode else dev32(f) for m, f in enumerate(F)], out)
        # CSF rounds nothing in between either: the per-fiber sum stays in double registers
        check(out, want, norm, f"mttkrp fp32 R={R}")


@pytest.mark.parametrize("attr", [(CN, S, S), (CU, CU, CU)])
def test_mttkrp_fp32_every_mode_of_a_fixed_tensor(attr):
    dims = (50, 40, 30)
    c, v = _coo(dims, 6000, 2)
    X = upload32(oracle.pack(c, v, dims, (0, 1, 2), attr))
    for R in (1, 5, 16):
        F = [f32(synth.random_dense((d, R), 2, 60 + m).numpy()) for m, d in enumerate(dims)]
        for mode in range(3):
            want, norm = oracle.mttkrp(c, v, dims, mode, F)
            out = torch.full((dims[mode], R), float("nan"), dtype=torch.float32, device="cuda")
            comet.mttkrp(X, mode, [None if m == mode else dev32(f) for m, f in enumerate(F)], out)
            check(out, want, norm, f"mttkrp fp32 mode {mode} R={R}")


@pytest.mark.parametrize("attr,order", [((D, CU), 2), ((CU, CU), 2), ((CN, S), 2), ((CU, CU, CU), 3), ((CN, S, S), 3)])
def test_pack_fp32_bit_exact(attr, order):
    dims = (300, 200) if order == 2 else (50, 40, 30)
    c, v = _coo(dims, 5000, 21)
    mode_order = tuple(range(order))
    want = oracle.pack(c, v, dims, mode_order, attr)
    T = comet.pack([dev(x, torch.int32) for x in c], dev32(v), dims, mode_order, attr)
    comet.validate(T)
    assert T.val.dtype == torch.float32
    assert np.array_equal(T.val.cpu().numpy().view(np.int32), want.val.astype(np.float32).view(np.int32))
    for l in range(order):
        assert_equal_arrays(T.pos(l), want.pos[l], f"pos{l}")
        assert_equal_arrays(T.crd(l), want.crd[l], f"crd{l}")


@pytest.mark.parametrize("config", [1, 2, 3, 4, 5])
def test_scaled_workloads_fp32(config, seg_dot_path):
    """The five benchmark workloads at 1/64 scale with float32 values, packed on the device."""
    case = synth.make(config, scale=1 / 64)
    c, v = [x.numpy() for x in case.coords], f32(case.val.numpy())
    dc = [x.cuda() for x in case.coords]
    dv = dev32(v)
    d32 = {k: f32(t.numpy()) for k, t in case.dense.items()}
    if config == 1:
        want, norm = oracle.spmv(c, v, case.dims, d32["x"])
        A = comet.pack(dc, dv, case.dims, (0, 1), (D, CU))
        check(comet.spmv(A, dev32(d32["x"])), want, norm, "C1 fp32")
    elif config == 2:
        want, norm = oracle.spmm(c, v, case.dims, d32["B"])
        A = comet.pack(dc, dv, case.dims, (0, 1), (D, CU))
        check(comet.spmm(A, dev32(d32["B"])), want, norm, "C2 fp32")
    elif config == 3:
        _, want, norm = oracle.ttv(c, v, case.dims, 2, d32["v"])
        X = comet.pack(dc, dv, case.dims, (0, 1, 2), (CU, CU, CU))
        check(comet.ttv(X, 2, dev32(d32["v"])).val, want, norm, "C3 fp32")
    elif config == 4:
        _, want, norm = oracle.ttm(c, v, case.dims, 2, d32["U"])
        X = comet.pack(dc, dv, case.dims, (0, 1, 2), (CU, CU, CU))
        check(comet.ttm(X, 2, dev32(d32["U"])).val.reshape(-1, case.R), want, norm, "C4 fp32")
    else:
        F = [None, d32["B"], d32["C"]]
        want, norm = oracle.mttkrp(c, v, case.dims, 0, F)
        Fd = [None, dev32(d32["B"]), dev32(d32["C"])]
        for attr in [(CN, S, S), (CU, CU, CU)]:
            X = comet.pack(dc, dv, case.dims, (0, 1, 2), attr)
            check(comet.mttkrp(X, 0, Fd), want, norm, f"C5 fp32 {attr}")


def test_mixed_value_types_are_refused():
    c, v = _coo((30, 20), 100, 2)
    A32 = upload32(oracle.pack(c, v, (30, 20), (0, 1), (D, CU)))
    with pytest.raises(TypeError):
        comet.spmv(A32, torch.ones(20, dtype=torch.float64, device="cuda"))
    with pytest.raises(TypeError):
        comet.spmm(A32, torch.ones((20, 4), dtype=torch.float64, device="cuda"))
    with pytest.raises(TypeError):
        comet.pack([dev(x, torch.int32) for x in c], torch.ones(100, dtype=torch.float16, device="cuda"), (30, 20),
                   (0, 1), (D, CU))
    # a float32 output tensor passed to the fp64 numeric phase is caught by the library itself
    tc, tv = _coo((10, 9, 8), 200, 3)
    X64 = comet.pack([dev(x, torch.int32) for x in tc], dev(tv), (10, 9, 8), (0, 1, 2), (CU, CU, CU))
    X32 = comet.pack([dev(x, torch.int32) for x in tc], dev32(tv), (10, 9, 8), (0, 1, 2), (CU, CU, CU))
    Y32 = comet.ttv_symbolic(X32, 2)
    with pytest.raises(comet.CometError):
        comet.ttv(X64, 2, torch.ones(8, dtype=torch.float64, device="cuda"), Y32)
