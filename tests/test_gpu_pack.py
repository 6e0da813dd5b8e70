"""GPU parity of comet_pack: every level array must equal the oracle's bit for bit (int32 arrays as
integers, values as 64-bit patterns), for every supported attribute tuple, storage order and order."""
import numpy as np
import pytest
import torch

import oracle
import synth
from oracle import D, CU, CN, S

pytestmark = pytest.mark.gpu

comet = pytest.importorskip("paper_2102_05187_b200")
from gpu_util import assert_close, assert_equal_arrays, dev  # noqa: E402


@pytest.fixture(autouse=True)
def _need_gpu(cuda_device):
    yield


def _np(coords):
    return [c.numpy() for c in coords]


def check_pack(coords, val, dims, mode_order, attr):
    want = oracle.pack(_np(coords), val.numpy(), dims, mode_order, attr)
    got = comet.pack([c.cuda() for c in coords], val.cuda(), dims, mode_order, attr)
    assert got.order == len(dims) and got.nnz == len(val) and got.attr == tuple(attr)
    assert got.mode_order == tuple(mode_order) and got.dims == tuple(dims)
    for l in range(len(dims)):
        assert_equal_arrays(got.pos(l), want.pos[l], f"pos[{l}] {attr} {mode_order}")
        assert_equal_arrays(got.crd(l), want.crd[l], f"crd[{l}] {attr} {mode_order}")
    if val.dtype == torch.float32:
        assert got.val.dtype == torch.float32
        assert np.array_equal(got.val.cpu().numpy().view(np.int32), want.val.astype(np.float32).view(np.int32)), "val"
    else:
        assert_equal_arrays(got.val, want.val, "val")
    comet.validate(got)
    return got


@pytest.fixture(params=["default", "csr-histogram", "generic"])
def csr_path(request, monkeypatch):
    """[D,CU] matrices: the size-based choice, then the histogram path and the generic radix path forced."""
    monkeypatch.delenv("COMET_PACK_CSR", raising=False)
    if request.param == "csr-histogram":
        monkeypatch.setenv("COMET_PACK_CSR", "1")
    elif request.param == "generic":
        monkeypatch.setenv("COMET_PACK_CSR", "0")
    return request.param


FORMATS_2D = [(CN, S), (D, CU), (CU, CU)]
FORMATS_3D = [(CN, S, S), (CU, CU, CU), (D, CU, CU)]


@pytest.mark.parametrize("attr", FORMATS_2D)
@pytest.mark.parametrize("mode_order", [(0, 1), (1, 0)])
@pytest.mark.parametrize("dims,nnz,seed", [((7, 5), 12, 1), ((1, 9), 4, 2), ((9, 1), 4, 3), ((6, 6), 36, 4),
                                           ((8, 8), 1, 5), ((8, 8), 0, 6), ((300, 200), 5000, 7),
                                           ((5000, 3), 9000, 8), ((3, 70000), 20000, 9), ((1, 1), 1, 10)])
def test_pack_matrices(attr, mode_order, dims, nnz, seed, csr_path):
    if attr != (D, CU) and csr_path != "default":
        pytest.skip("the path choice only exists for [D,CU]")
    coords, val = synth.random_coo(dims, nnz, seed)
    check_pack(coords, val, dims, mode_order, attr)


@pytest.mark.parametrize("mode_order", [(0, 1), (1, 0)])
@pytest.mark.parametrize("dims,nnz,seed", [((40, 3000), 30000, 1),      # rows of ~750: the shared-memory network
                                           ((6, 9000), 30000, 2),       # rows of ~5000: the shared-memory radix sort
                                           ((3, 12288), 36864, 3),      # full rows of exactly the longest length handled
                                           ((2, 40000), 50000, 4),      # rows of 25000: handed to the generic path
                                           ((2000, 2100), 60000, 5),    # every class of short row
                                           ((70, 33), 2310, 6)])        # rows of exactly 33: the first mid length
def test_pack_csr_row_length_classes(mode_order, dims, nnz, seed, csr_path):
    d = dims if mode_order == (0, 1) else (dims[1], dims[0])
    coords, val = synth.random_coo(dims, nnz, seed)
    if mode_order == (1, 0):
        coords = [coords[1], coords[0]]
    check_pack(coords, val, d, mode_order, (D, CU))
    check_pack(coords, val.float(), d, mode_order, (D, CU))


def test_pack_csr_histogram_path_reports_errors(monkeypatch):
    monkeypatch.setenv("COMET_PACK_CSR", "1")
    r = torch.tensor([0, 1, 1, 5], dtype=torch.int32, device="cuda")
    c = torch.tensor([0, 1, 1, 2], dtype=torch.int32, device="cuda")
    v = torch.ones(4, dtype=torch.float64, device="cuda")
    with pytest.raises(comet.CometError) as e:
        comet.pack([r[:3], c[:3]], v[:3], (4, 4), (0, 1), (D, CU))
    assert comet.binding.STATUS_NAMES[e.value.status] == "COMET_ERR_DUPLICATE_COORD"
    with pytest.raises(comet.CometError) as e:
        comet.pack([r, c], v, (4, 4), (0, 1), (D, CU))
    assert comet.binding.STATUS_NAMES[e.value.status] == "COMET_ERR_COORD_OUT_OF_RANGE"
    # duplicates inside a long row (the shared-memory sorts check neighbours too)
    g = np.random.default_rng(1)
    cols = torch.from_numpy(g.permutation(9000)[:5000].astype(np.int32)).cuda()
    cols[4999] = cols[17]
    rows = torch.zeros(5000, dtype=torch.int32, device="cuda")
    with pytest.raises(comet.CometError) as e:
        comet.pack([rows, cols], torch.ones(5000, dtype=torch.float64, device="cuda"), (1, 9000), (0, 1), (D, CU))
    assert comet.binding.STATUS_NAMES[e.value.status] == "COMET_ERR_DUPLICATE_COORD"
    cols2 = torch.from_numpy(g.permutation(3000)[:700].astype(np.int32)).cuda()
    cols2[699] = cols2[5]
    with pytest.raises(comet.CometError) as e:
        comet.pack([torch.zeros(700, dtype=torch.int32, device="cuda"), cols2], torch.ones(700, dtype=torch.float64, device="cuda"),
                   (1, 3000), (0, 1), (D, CU))
    assert comet.binding.STATUS_NAMES[e.value.status] == "COMET_ERR_DUPLICATE_COORD"


@pytest.mark.parametrize("attr", FORMATS_3D)
@pytest.mark.parametrize("mode_order", [(0, 1, 2), (1, 0, 2), (2, 1, 0), (1, 2, 0)])
@pytest.mark.parametrize("dims,nnz,seed", [((4, 5, 6), 30, 1), ((3, 1, 7), 9, 2), ((5, 5, 5), 125, 3),
                                           ((6, 4, 3), 0, 4), ((9, 8, 7), 1, 5), ((60, 50, 40), 20000, 6),
                                           ((2000, 3, 1000), 30000, 7)])
def test_pack_tensors(attr, mode_order, dims, nnz, seed):
    coords, val = synth.random_coo(dims, nnz, seed)
    check_pack(coords, val, dims, mode_order, attr)


def test_pack_order4():
    dims = (9, 8, 7, 6)
    coords, val = synth.random_coo(dims, 1500, 11)
    for attr in [(CU, CU, CU, CU), (CN, S, S, S), (D, CU, CU, CU)]:
        check_pack(coords, val, dims, (0, 1, 2, 3), attr)
        check_pack(coords, val, dims, (3, 1, 0, 2), attr)


def test_pack_large_extents_use_many_radix_passes():
    dims = (1_000_000, 500_000, 200_000)            # 57 key bits: 8 passes
    coords, val = synth.random_coo(dims, 60_000, 12)
    check_pack(coords, val, dims, (0, 1, 2), (CU, CU, CU))
    check_pack(coords, val, dims, (0, 1, 2), (CN, S, S))


@pytest.mark.parametrize("config,attr", [(1, (D, CU)), (2, (D, CU)), (3, (CU, CU, CU)), (4, (CU, CU, CU)),
                                         (5, (CN, S, S)), (5, (CU, CU, CU))])
def test_pack_scaled_workloads(config, attr):
    case = synth.make(config, scale=1 / 64)
    order = tuple(range(len(case.dims)))
    check_pack(case.coords, case.val, case.dims, order, attr)


def test_shuffled_input_gives_identical_arrays():
    dims = (50, 40, 30)
    coords, val = synth.random_coo(dims, 8000, 21)
    a = comet.pack([c.cuda() for c in coords], val.cuda(), dims, (0, 1, 2), (CU, CU, CU))
    p = torch.randperm(len(val), generator=torch.Generator().manual_seed(3))
    b = comet.pack([c[p].cuda() for c in coords], val[p].cuda(), dims, (0, 1, 2), (CU, CU, CU))
    for l in range(3):
        assert torch.equal(a.pos(l), b.pos(l)) and torch.equal(a.crd(l), b.crd(l))
    assert torch.equal(a.val, b.val)


def test_rejected_inputs():
    i = torch.tensor([0, 0], dtype=torch.int32).cuda()
    j = torch.tensor([1, 1], dtype=torch.int32).cuda()
    v = torch.ones(2, dtype=torch.float64).cuda()
    for attr in [(D, CU), (CN, S), (CU, CU)]:
        with pytest.raises(comet.CometError) as e:
            comet.pack([i, j], v, (2, 2), (0, 1), attr)
        assert e.value.status == -4                      # duplicate coordinate
    with pytest.raises(comet.CometError) as e:
        comet.pack([i, torch.tensor([1, 2], dtype=torch.int32).cuda()], v, (2, 2), (0, 1), (D, CU))
    assert e.value.status == -3                          # out of range
    with pytest.raises(comet.CometError) as e:
        comet.pack([i, torch.tensor([-1, 0], dtype=torch.int32).cuda()], v, (2, 2), (0, 1), (D, CU))
    assert e.value.status == -3
    for bad in [(CU, D), (CU, CN), (CU, S), (S, S), (D, D)]:
        with pytest.raises(comet.CometError) as e:
            comet.pack([i, j], v, (2, 2), (0, 1), bad)
        assert e.value.status == -2
    with pytest.raises(comet.CometError) as e:
        comet.pack([i, j], v, (2, 2), (0, 0), (D, CU))
    assert e.value.status == -1
    # the handle is still usable afterwards
    ok = comet.pack([torch.tensor([0, 1], dtype=torch.int32).cuda(), j], v, (2, 2), (0, 1), (D, CU))
    assert ok.pos(1).tolist() == [0, 1, 2]


def test_validate_catches_broken_descriptors():
    dims = (30, 20)
    coords, val = synth.random_coo(dims, 200, 5)
    pk = oracle.pack(_np(coords), val.numpy(), dims, (0, 1), (D, CU))
    def build(pos1, crd1):
        return comet.SpTensor.from_arrays(dims, (0, 1), (D, CU), [dev(pk.pos[0], torch.int32), dev(pos1, torch.int32)],
                                          [None, dev(crd1, torch.int32)], dev(pk.val))
    comet.validate(build(pk.pos[1], pk.crd[1]))
    bad_pos = pk.pos[1].copy(); bad_pos[5] = bad_pos[6] + 1
    bad_crd = pk.crd[1].copy(); bad_crd[3] = dims[1]
    unsorted = pk.crd[1].copy()
    row = int(np.argmax(np.diff(pk.pos[1]) >= 2))
    a = pk.pos[1][row]; unsorted[a], unsorted[a + 1] = unsorted[a + 1], unsorted[a]
    for pos1, crd1 in [(bad_pos, pk.crd[1]), (pk.pos[1], bad_crd), (pk.pos[1], unsorted)]:
        with pytest.raises(comet.CometError) as e:
            comet.validate(build(pos1, crd1))
        assert e.value.status == -10


def test_pack_then_contract_end_to_end():
    case = synth.make(4, scale=1 / 64)
    X = comet.pack([c.cuda() for c in case.coords], case.val.cuda(), case.dims, (0, 1, 2), (CU, CU, CU))
    Y = comet.ttm(X, 2, case.dense["U"].cuda())
    _, want, norm = oracle.ttm(_np(case.coords), case.val.numpy(), case.dims, 2, case.dense["U"].numpy())
    assert_close(Y.val.reshape(-1, case.R), want, norm, what="pack+ttm")


# ----------------------------------------------------------------------------- COMET_PACK_SUM_DUPLICATES
def _with_duplicates(dims, n, seed):
    """n entries over few cells (many repeats), values of very different magnitudes so that the order of the
    additions shows in the last bits."""
    g = np.random.default_rng(seed)
    coords = [torch.from_numpy(g.integers(0, d, n).astype(np.int32)) for d in dims]
    val = torch.from_numpy(g.standard_normal(n) * 10.0 ** g.integers(-8, 9, n))
    return coords, val


@pytest.mark.parametrize("dims,n,attr,mode_order", [
    ((7, 9), 400, (D, CU), (0, 1)), ((7, 9), 400, (CU, CU), (1, 0)), ((7, 9), 400, (CN, S), (0, 1)),
    ((40, 30), 20000, (D, CU), (0, 1)), ((6, 5, 4), 3000, (CU, CU, CU), (2, 0, 1)), ((6, 5, 4), 3000, (CN, S, S), (0, 1, 2)),
    ((30, 20, 10), 50000, (D, CU, CU), (1, 2, 0)), ((5, 4, 3, 2), 4000, (CU, CU, CU, CU), (3, 2, 1, 0)),
    ((1, 1), 1000, (D, CU), (0, 1)), ((300, 200), 500, (D, CU), (0, 1))])
def test_pack_sum_duplicates_bit_exact(dims, n, attr, mode_order):
    coords, val = _with_duplicates(dims, n, 17)
    want = oracle.pack(_np(coords), val.numpy(), dims, mode_order, attr, sum_duplicates_first=True)
    got = comet.pack([c.cuda() for c in coords], val.cuda(), dims, mode_order, attr, sum_duplicates=True)
    assert got.nnz == len(want.val) and got.nnz <= n
    for l in range(len(dims)):
        assert_equal_arrays(got.pos(l), want.pos[l], f"pos[{l}]")
        assert_equal_arrays(got.crd(l), want.crd[l], f"crd[{l}]")
    assert_equal_arrays(got.val, want.val, "merged values")        # same additions in the same order: same bits
    comet.validate(got)
    with pytest.raises(comet.CometError) as e:                     # without the flag the same input is refused
        comet.pack([c.cuda() for c in coords], val.cuda(), dims, mode_order, attr)
    assert comet.binding.STATUS_NAMES[e.value.status] == "COMET_ERR_DUPLICATE_COORD"


def test_pack_sum_duplicates_is_a_no_op_on_distinct_cells_and_handles_empty_and_fp32():
    dims = (60, 50, 40)
    coords, val = synth.random_coo(dims, 20000, 6)
    a = comet.pack([c.cuda() for c in coords], val.cuda(), dims, (0, 1, 2), (CU, CU, CU))
    b = comet.pack([c.cuda() for c in coords], val.cuda(), dims, (0, 1, 2), (CU, CU, CU), sum_duplicates=True)
    assert a.nnz == b.nnz and torch.equal(a.val, b.val)
    for l in range(3):
        assert torch.equal(a.pos(l), b.pos(l)) and torch.equal(a.crd(l), b.crd(l))
    e = comet.pack([torch.zeros(0, dtype=torch.int32, device="cuda")] * 2, torch.zeros(0, dtype=torch.float64, device="cuda"),
                   (4, 4), (0, 1), (D, CU), sum_duplicates=True)
    assert e.nnz == 0 and e.pos(1).tolist() == [0, 0, 0, 0, 0]
    dc, dv = _with_duplicates((7, 9), 400, 3)
    v32 = dv.float()
    want = oracle.pack(_np(dc), v32.double().numpy(), (7, 9), (0, 1), (D, CU), sum_duplicates_first=True)
    got = comet.pack([c.cuda() for c in dc], v32.cuda(), (7, 9), (0, 1), (D, CU), sum_duplicates=True)
    assert got.val.dtype == torch.float32
    assert np.array_equal(got.val.cpu().numpy(), want.val.astype(np.float32))   # summed in double, rounded once


@pytest.mark.parametrize("dtype", [torch.float64, torch.float32])
def test_pack_of_extent_one_tensors_and_of_keys_that_fill_a_whole_number_of_passes(dtype):
    """Keys of zero bits (every extent 1: no sort pass runs), of exactly 8 and 16 bits (the last pass is a full
    digit), and of 9 bits (a last pass over a single bit), fp64 values (gathered through the sorted indices) and
    fp32 ones (carried through the sort)."""
    one = [torch.zeros(1, dtype=torch.int32, device="cuda")] * 3
    t = comet.pack(one, torch.tensor([2.5], dtype=dtype, device="cuda"), (1, 1, 1), (0, 1, 2), (CU, CU, CU))
    assert t.nnz == 1 and t.val.tolist() == [2.5] and t.crd(2).tolist() == [0]
    dup = [torch.zeros(3, dtype=torch.int32, device="cuda")] * 2
    s = comet.pack(dup, torch.tensor([1.0, 2.0, 4.0], dtype=dtype, device="cuda"), (1, 1), (0, 1), (D, CU), sum_duplicates=True)
    assert s.nnz == 1 and s.val.tolist() == [7.0]
    for dims in [(16, 16), (256, 256), (32, 16)]:
        coords, val = synth.random_coo(dims, min(200, dims[0] * dims[1] // 2), 9)
        val = val.to(dtype)
        want = oracle.pack(_np(coords), val.double().numpy(), dims, (1, 0), (D, CU))
        got = comet.pack([c.cuda() for c in coords], val.cuda(), dims, (1, 0), (D, CU))
        assert got.pos(1).tolist() == want.pos[1].tolist() and got.crd(1).tolist() == want.crd[1].tolist()
        assert np.array_equal(got.val.double().cpu().numpy(), want.val)


def test_pack_csr_histogram_flag_gives_the_same_tensor():
    dims = (300, 200)
    coords, val = synth.random_coo(dims, 5000, 7)
    a = comet.pack([c.cuda() for c in coords], val.cuda(), dims, (0, 1), (D, CU))
    b = comet.pack([c.cuda() for c in coords], val.cuda(), dims, (0, 1), (D, CU), csr_histogram=True)
    assert torch.equal(a.val, b.val) and torch.equal(a.pos(1), b.pos(1)) and torch.equal(a.crd(1), b.crd(1))
    c3 = comet.pack([c.cuda() for c in coords], val.cuda(), dims, (0, 1), (CU, CU), csr_histogram=True)   # ignored here
    assert c3.attr == (CU, CU)


def test_pack_ex_rejects_unknown_flags():
    import ctypes as C
    h = comet.default_handle()
    out = comet.binding.SpTensorStruct()
    dims = (C.c_int64 * 2)(2, 2)
    crd = (C.c_void_p * 2)(0, 0)
    mo = (C.c_int32 * 2)(0, 1)
    at = (C.c_int32 * 2)(D, CU)
    st = h.lib.comet_pack_ex(h._h, C.c_int32(2), dims, C.c_int64(0), crd, None, C.c_int(0), mo, at, C.c_uint32(12), None,
                             C.byref(out))
    assert st == -1
