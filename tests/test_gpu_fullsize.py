"""Full-size checks, in the launch configuration bench.py times: every workload at scale 1.

Packing: the packed arrays are expanded back to coordinate lists (Table 1's loops, vectorised) and must
equal the lexicographically sorted input bit for bit; pos arrays must be monotone and end at the next
level's length. Contractions: a seeded sample of output rows / fibers is recomputed one by one by the
CPU oracle over the raw COO entries and compared with the normalised fp64 tolerance.
"""
import numpy as np
import pytest
import torch

import oracle
import synth
from oracle import D, CU, CN, S

pytestmark = pytest.mark.gpu

comet = pytest.importorskip("paper_2102_05187_b200")
from gpu_util import FP64_TOL, assert_close  # noqa: E402

SAMPLES = 48


@pytest.fixture(autouse=True)
def _need_gpu(cuda_device):
    yield


def _expand(pos, n_children):
    """parent index of every child position from a pos array (the CU loop of Table 1, vectorised)."""
    counts = (pos[1:] - pos[:-1]).long()
    assert int(counts.min()) >= 0 and int(pos[0]) == 0 and int(pos[-1]) == n_children
    return torch.repeat_interleave(torch.arange(counts.numel(), device=pos.device), counts)


def check_packed_against_sorted_input(case, T, mode_order, attr):
    """Rebuild the coordinate list from the packed levels and compare with the sorted input."""
    n = case.nnz
    key = torch.zeros(n, dtype=torch.int64, device="cuda")
    for m in mode_order:
        key = key * case.dims[m] + case.coords[m].long()
    order = torch.sort(key, stable=True).indices
    want = [case.coords[m][order] for m in mode_order]
    assert torch.equal(T.val, case.val[order]), "values are not the input values in sorted order"
    # walk from the leaf upwards: position of each leaf entry at each level
    levels = len(mode_order)
    positions = [None] * levels
    positions[levels - 1] = torch.arange(n, device="cuda")
    for l in range(levels - 1, 0, -1):
        a = attr[l]
        if a == CU:
            up = _expand(T.pos(l), T.c.crd_len[l])           # parent position of every node of level l
            positions[l - 1] = up[positions[l]]
        else:                                                # S: same position as the level above
            positions[l - 1] = positions[l]
    for l in range(levels):
        a = attr[l]
        if a == D:
            got = positions[l].to(torch.int32)               # under a dense root the position IS the coordinate
            assert T.pos(l).tolist() == [case.dims[mode_order[l]]]
        else:
            crd = T.crd(l)
            assert int(crd.min()) >= 0 and int(crd.max()) < case.dims[mode_order[l]]
            got = crd[positions[l]]
            if a == CN:
                assert T.pos(l).tolist() == [0, n]
            if a == CU and l == 0:
                assert T.pos(0).tolist() == [0, T.c.crd_len[0]]
        assert torch.equal(got, want[l]), f"level {l}: coordinates differ from the sorted input"
    # CU coordinates strictly ascend inside each parent: follows from equality with the sorted distinct input
    return order


def sample_rows(n_rows, seed, always=()):
    g = np.random.default_rng(seed)
    rows = set(int(r) for r in g.integers(0, n_rows, SAMPLES))
    rows.update(int(r) for r in always if 0 <= r < n_rows)
    return np.array(sorted(rows), dtype=np.int64)


def host(case):
    return [c.cpu().numpy() for c in case.coords], case.val.cpu().numpy()


def test_full_c1_spmv():
    case = synth.make(1, device="cuda")
    A = comet.pack(case.coords, case.val, case.dims, (0, 1), (D, CU))
    check_packed_against_sorted_input(case, A, (0, 1), (D, CU))
    y = comet.spmv(A, case.dense["x"])
    c, v = host(case)
    want, norm = oracle.spmv(c, v, case.dims, case.dense["x"].cpu().numpy())      # small enough for every row
    assert_close(y, want, norm, what="C1 spmv")


def test_full_c2_spmm():
    case = synth.make(2, device="cuda")
    A = comet.pack(case.coords, case.val, case.dims, (0, 1), (D, CU))
    check_packed_against_sorted_input(case, A, (0, 1), (D, CU))
    C = comet.spmm(A, case.dense["B"])
    lengths = torch.bincount(case.coords[0].long(), minlength=case.dims[0])
    heavy = torch.topk(lengths, 4).indices.tolist()                                # rows that span many tiles
    rows = sample_rows(case.dims[0], 2, always=heavy + [0, case.dims[0] - 1])
    c, v = host(case)
    want, norm = oracle.spmm(c, v, case.dims, case.dense["B"].cpu().numpy(), rows=rows)
    rel = assert_close(C[torch.from_numpy(rows).cuda()], want, norm, what="C2 spmm")
    print(f"C2 worst normalised error {rel:.2e}")


def test_full_c3_ttv():
    case = synth.make(3, device="cuda")
    X = comet.pack(case.coords, case.val, case.dims, (0, 1, 2), (CU, CU, CU))
    check_packed_against_sorted_input(case, X, (0, 1, 2), (CU, CU, CU))
    Y = comet.ttv(X, 2, case.dense["v"])
    F = X.c.crd_len[1]
    fib = sample_rows(F, 3, always=[0, F - 1])
    # the (i, j) key of sampled fiber f: crd1[f] and the slice that holds it
    slice_of = _expand(X.pos(1), F)
    fi = X.crd(0)[slice_of[torch.from_numpy(fib).cuda()]].long()
    fj = X.crd(1)[torch.from_numpy(fib).cuda()].long()
    keys = (fi * case.dims[1] + fj).cpu().numpy()
    assert np.all(np.diff(keys) > 0)
    c, v = host(case)
    _, want, norm = oracle.ttv(c, v, case.dims, 2, case.dense["v"].cpu().numpy(), keys=keys)
    rel = assert_close(Y.val[torch.from_numpy(fib).cuda()], want, norm, what="C3 ttv")
    print(f"C3 worst normalised error {rel:.2e}")
    # output structure: CSR over (I, J) whose rows are the slices
    pos = Y.pos(1)
    assert pos.numel() == case.dims[0] + 1 and int(pos[-1]) == F and bool((pos[1:] >= pos[:-1]).all())
    assert torch.equal(Y.crd(1), X.crd(1))


def test_full_c4_ttm():
    case = synth.make(4, device="cuda")
    X = comet.pack(case.coords, case.val, case.dims, (0, 1, 2), (CU, CU, CU))
    check_packed_against_sorted_input(case, X, (0, 1, 2), (CU, CU, CU))
    Y = comet.ttm(X, 2, case.dense["U"])
    F = X.c.crd_len[1]
    fib = sample_rows(F, 4, always=[0, F - 1])
    sel = torch.from_numpy(fib).cuda()
    slice_of = _expand(X.pos(1), F)
    keys = (X.crd(0)[slice_of[sel]].long() * case.dims[1] + X.crd(1)[sel].long()).cpu().numpy()
    c, v = host(case)
    _, want, norm = oracle.ttm(c, v, case.dims, 2, case.dense["U"].cpu().numpy(), keys=keys)
    rel = assert_close(Y.val.reshape(F, case.R)[sel], want, norm, what="C4 ttm")
    print(f"C4 worst normalised error {rel:.2e}")


@pytest.mark.parametrize("attr", [(CN, S, S), (CU, CU, CU)])
def test_full_c5_mttkrp(attr):
    case = synth.make(5, device="cuda")
    X = comet.pack(case.coords, case.val, case.dims, (0, 1, 2), attr)
    check_packed_against_sorted_input(case, X, (0, 1, 2), attr)
    Fd = [None, case.dense["B"], case.dense["C"]]
    out = torch.full((case.dims[0], case.R), float("nan"), dtype=torch.float64, device="cuda")
    comet.mttkrp(X, 0, Fd, out)
    assert not bool(torch.isnan(out).any()), "an output row was not written"
    counts = torch.bincount(case.coords[0].long(), minlength=case.dims[0])
    heavy = torch.topk(counts, 4).indices.tolist()                                 # slices spanning thousands of tiles
    empty = torch.nonzero(counts == 0)[:4, 0].tolist()
    rows = sample_rows(case.dims[0], 5, always=heavy + empty + [0, case.dims[0] - 1])
    del X
    c, v = host(case)
    want, norm = oracle.mttkrp(c, v, case.dims, 0, [None, Fd[1].cpu().numpy(), Fd[2].cpu().numpy()], rows=rows)
    rel = assert_close(out[torch.from_numpy(rows).cuda()], want, norm, what=f"C5 mttkrp {attr}")
    print(f"C5 {attr} worst normalised error {rel:.2e}")
    assert bool((out[counts == 0] == 0).all())                                     # rows without entries are +0


@pytest.mark.parametrize("attr", [(CN, S, S), (CU, CU, CU)])
@pytest.mark.parametrize("mode", [1, 2])
def test_full_c5_mttkrp_non_root_modes(attr, mode):
    """Modes 1 and 2 on the tensor packed with mode 0 first (atomic accumulation), sampled rows."""
    case = synth.make(5, device="cuda")
    X = comet.pack(case.coords, case.val, case.dims, (0, 1, 2), attr)
    R = case.R
    F = [synth.random_dense((d, R), case.seed, 70 + m, device="cuda") for m, d in enumerate(case.dims)]
    out = torch.full((case.dims[mode], R), float("nan"), dtype=torch.float64, device="cuda")
    comet.mttkrp(X, mode, [None if m == mode else f for m, f in enumerate(F)], out)
    assert not bool(torch.isnan(out).any()), "an output row was not written"
    counts = torch.bincount(case.coords[mode].long(), minlength=case.dims[mode])
    heavy = torch.topk(counts, 4).indices.tolist()
    empty = torch.nonzero(counts == 0)[:4, 0].tolist()
    rows = sample_rows(case.dims[mode], 5, always=heavy + empty + [0, case.dims[mode] - 1])
    del X
    c, v = host(case)
    want, norm = oracle.mttkrp(c, v, case.dims, mode, [None if m == mode else f.cpu().numpy() for m, f in enumerate(F)],
                               rows=rows)
    rel = assert_close(out[torch.from_numpy(rows).cuda()], want, norm, what=f"C5 mttkrp mode {mode} {attr}")
    print(f"C5 mode {mode} {attr} worst normalised error {rel:.2e}")
    assert bool((out[counts == 0] == 0).all())


def test_full_c3_c4_from_sorted_coo_equal_the_csf_results():
    """[CN,S,S] inputs at full size: the derived fibers must reproduce the CSF tensor's structure, and the
    values (same kernels, same boundaries) must be bit-identical to the CSF results, which the tests above
    check against the oracle."""
    for cfg in (3, 4):
        case = synth.make(cfg, device="cuda")
        Xs = comet.pack(case.coords, case.val, case.dims, (0, 1, 2), (CU, CU, CU))
        Xc = comet.pack(case.coords, case.val, case.dims, (0, 1, 2), (CN, S, S))
        if cfg == 3:
            Ys, Yc = comet.ttv(Xs, 2, case.dense["v"]), comet.ttv(Xc, 2, case.dense["v"])
        else:
            Ys, Yc = comet.ttm(Xs, 2, case.dense["U"]), comet.ttm(Xc, 2, case.dense["U"])
        assert Yc.c.nnz == Ys.c.nnz and Yc.attr == Ys.attr and Yc.dims == Ys.dims
        for l in range(2):
            assert torch.equal(Yc.pos(l), Ys.pos(l)) and torch.equal(Yc.crd(l), Ys.crd(l))
        assert torch.equal(Yc.val, Ys.val)
        del Xs, Xc, Ys, Yc, case
        torch.cuda.empty_cache()


def test_hypersparse_matrix_csr_dcsr_coo():
    """A second workload shape: 67,108,864 x 1,048,576 with 4,194,304 uniform distinct entries (94 % of the
    rows are empty), the setting in which the paper stores both dimensions compressed. All three matrix
    formats must give the oracle's rows, +0 in the empty rows, and DCSR must be the smallest index."""
    dims, nnz, R = (1 << 26, 1 << 20), 1 << 22, 8
    coords, val = synth.random_coo(dims, nnz, 77, device="cuda")
    x = synth.random_dense((dims[1],), 77, device="cuda")
    B = synth.random_dense((dims[1], R), 77, 51, device="cuda")
    counts = torch.bincount(coords[0].long(), minlength=dims[0])
    stored = torch.nonzero(counts)[:, 0]
    picks = stored[torch.linspace(0, stored.numel() - 1, 40, device="cuda").long()].tolist()
    rows = sample_rows(dims[0], 9, always=picks + [0, dims[0] - 1])
    c, v = [t.cpu().numpy() for t in coords], val.cpu().numpy()
    want_y, norm_y = oracle.spmv(c, v, dims, x.cpu().numpy(), rows=rows)
    want_c, norm_c = oracle.spmm(c, v, dims, B.cpu().numpy(), rows=rows)
    sel = torch.from_numpy(rows).cuda()
    index_bytes = {}
    for name, attr in (("csr", (D, CU)), ("dcsr", (CU, CU)), ("coo", (CN, S))):
        A = comet.pack(coords, val, dims, (0, 1), attr)
        index_bytes[name] = 4 * sum(A.c.pos_len[l] + A.c.crd_len[l] for l in range(2))
        y = torch.full((dims[0],), float("nan"), dtype=torch.float64, device="cuda")
        comet.spmv(A, x, y)
        assert_close(y[sel], want_y, norm_y, what=f"hypersparse spmv {name}")
        assert bool((y[counts == 0] == 0).all())
        del y
        C = torch.full((dims[0], R), float("nan"), dtype=torch.float64, device="cuda")
        comet.spmm(A, B, C)
        assert_close(C[sel], want_c, norm_c, what=f"hypersparse spmm {name}")
        assert bool((C[counts == 0] == 0).all())
        del C, A
        torch.cuda.empty_cache()
    assert index_bytes["dcsr"] < index_bytes["csr"] / 5


def test_large_matrix_268m_entries():
    """Sizes well beyond the benchmark's: 268,435,456 entries in a 1,048,576^2 matrix (positions and merge-list
    indices in the 2^28..2^29 range). Packing is checked against the sorted input, SpMV on sampled rows."""
    dims, nnz = (1 << 20, 1 << 20), 1 << 28
    coords, val = synth.random_coo(dims, nnz, 91, device="cuda")

    class _Case:
        pass
    case = _Case()
    case.nnz, case.dims, case.coords, case.val = nnz, dims, coords, val
    A = comet.pack(coords, val, dims, (0, 1), (D, CU))
    check_packed_against_sorted_input(case, A, (0, 1), (D, CU))
    x = synth.random_dense((dims[1],), 91, device="cuda")
    y = torch.full((dims[0],), float("nan"), dtype=torch.float64, device="cuda")
    comet.spmv(A, x, y)
    assert not bool(torch.isnan(y).any())
    rows = sample_rows(dims[0], 13, always=[0, dims[0] - 1])
    c, v = [t.cpu().numpy() for t in coords], val.cpu().numpy()
    del A, coords, val
    torch.cuda.empty_cache()
    want, norm = oracle.spmv(c, v, dims, x.cpu().numpy(), rows=rows)
    rel = assert_close(y[torch.from_numpy(rows).cuda()], want, norm, what="268M-entry spmv")
    print(f"268M entries: worst normalised error {rel:.2e}")


def test_full_fp32_c2_spmm_and_c5_coo_mttkrp():
    """fp32 values at full size (the long-row path of SpMM and the tiled COO MTTKRP): the oracle is fed the same
    float32 numbers widened to double; both the stated 1e-5 tolerance and the rounding bound of two float roundings
    (the store and one carry addition) must hold."""
    case = synth.make(2, device="cuda")
    v32, B32 = case.val.float(), case.dense["B"].float()
    A = comet.pack(case.coords, v32, case.dims, (0, 1), (D, CU))
    C = torch.full((case.dims[0], case.R), float("nan"), dtype=torch.float32, device="cuda")
    comet.spmm(A, B32, C)
    lengths = torch.bincount(case.coords[0].long(), minlength=case.dims[0])
    rows = sample_rows(case.dims[0], 12, always=torch.topk(lengths, 4).indices.tolist() + [0, case.dims[0] - 1])
    c = [x.cpu().numpy() for x in case.coords]
    want, norm = oracle.spmm(c, v32.double().cpu().numpy(), case.dims, B32.double().cpu().numpy(), rows=rows)
    got = C[torch.from_numpy(rows).cuda()].double()
    assert_close(got, want, norm, tol=1e-5, what="C2 spmm fp32")
    assert_close(got, want, norm, tol=3 * 2.0 ** -24, what="C2 spmm fp32 (rounding bound)")
    del A, C, case
    torch.cuda.empty_cache()

    case = synth.make(5, device="cuda")
    v32 = case.val.float()
    Fd = [None, case.dense["B"].float(), case.dense["C"].float()]
    X = comet.pack(case.coords, v32, case.dims, (0, 1, 2), (CN, S, S))
    out = torch.full((case.dims[0], case.R), float("nan"), dtype=torch.float32, device="cuda")
    comet.mttkrp(X, 0, Fd, out)
    counts = torch.bincount(case.coords[0].long(), minlength=case.dims[0])
    rows = sample_rows(case.dims[0], 15, always=torch.topk(counts, 4).indices.tolist() + [0, case.dims[0] - 1])
    del X
    c = [x.cpu().numpy() for x in case.coords]
    want, norm = oracle.mttkrp(c, v32.double().cpu().numpy(), case.dims, 0,
                               [None, Fd[1].double().cpu().numpy(), Fd[2].double().cpu().numpy()], rows=rows)
    got = out[torch.from_numpy(rows).cuda()].double()
    assert_close(got, want, norm, tol=1e-5, what="C5 coo mttkrp fp32")
    assert_close(got, want, norm, tol=3 * 2.0 ** -24, what="C5 coo mttkrp fp32 (rounding bound)")
