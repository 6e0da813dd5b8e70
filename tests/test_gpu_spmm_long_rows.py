"""GPU parity of the long-row path of comet_spmm (rows cut into column blocks, the tiles of a block processed
together so that the block of B stays in L2; the short rows by the general kernel, both in one launch).

The path switches itself on only for matrices with millions of entries and a B of hundreds of MB; here the
tuning variables force it on small matrices whose row lengths are built by hand: long rows at the first and the
last row, next to each other, next to empty rows, a row with exactly the threshold, a row whose columns all fall
into one block, and nothing but long rows. Every output element is compared with the CPU oracle."""
import numpy as np
import pytest
import torch

import oracle
import synth
from oracle import D, CU

pytestmark = pytest.mark.gpu

comet = pytest.importorskip("paper_2102_05187_b200")
from gpu_util import assert_close, dev, upload_packed  # noqa: E402


@pytest.fixture(autouse=True)
def _need_gpu(cuda_device):
    yield


@pytest.fixture
def force_long_rows(monkeypatch):
    def set_env(threshold=40, tile=32, piece=8, blocks=4, ctas=3, tile_items=37):
        monkeypatch.setenv("COMET_SPMM_LONG_MIN_NNZ", "1")
        monkeypatch.setenv("COMET_SPMM_LONG_MIN_B_MB", "0")
        monkeypatch.setenv("COMET_SPMM_LONG_ROW", str(threshold))
        monkeypatch.setenv("COMET_SPMM_LONG_TILE", str(tile))
        monkeypatch.setenv("COMET_SPMM_PIECE", str(piece))
        monkeypatch.setenv("COMET_SPMM_BLOCKS", str(blocks))
        monkeypatch.setenv("COMET_SPMM_LONG_CTAS", str(ctas))
        monkeypatch.setenv("COMET_TILE_ITEMS", str(tile_items))
    return set_env


def matrix_from_row_lengths(lengths, cols, seed, col_range=None):
    """COO entries (shuffled) of a matrix whose row i holds lengths[i] distinct columns."""
    rng = np.random.default_rng(seed)
    ri, ci = [], []
    for i, n in enumerate(lengths):
        lo, hi = col_range.get(i, (0, cols)) if col_range else (0, cols)
        ci.append(rng.choice(np.arange(lo, hi), size=n, replace=False))
        ri.append(np.full(n, i))
    ri = np.concatenate(ri).astype(np.int32)
    ci = np.concatenate(ci).astype(np.int32)
    perm = rng.permutation(ri.size)
    val = rng.uniform(-1, 1, ri.size)
    return [ri[perm], ci[perm]], val[perm]


def lengths_mixed(rows, seed):
    rng = np.random.default_rng(seed)
    ln = rng.integers(0, 6, rows)                       # short and empty rows
    ln[0] = 300                                         # long first row
    ln[1] = 0
    ln[2] = 0
    ln[5] = 40                                          # exactly the threshold
    ln[6] = 39                                          # one below it
    ln[7] = 41
    ln[20] = 500                                        # three long rows in a row
    ln[21] = 77
    ln[22] = 130
    ln[23] = 0
    ln[rows - 1] = 250                                  # long last row
    ln[rows // 2] = 64                                  # a long row confined to one block of columns (below)
    return ln


CASES = [("mixed", 400, 640), ("all-long", 30, 512), ("one-long-row", 1, 700), ("no-long-row", 300, 600)]


def build(kind, rows, cols, seed):
    if kind == "mixed":
        ln = lengths_mixed(rows, seed)
        rng_cols = {rows // 2: (cols // 4 + 3, cols // 2 - 5)}
    elif kind == "all-long":
        ln = np.random.default_rng(seed).integers(40, 400, rows)
        rng_cols = None
    elif kind == "one-long-row":
        ln = np.array([600])
        rng_cols = None
    else:
        ln = np.random.default_rng(seed).integers(0, 30, rows)
        rng_cols = None
    return matrix_from_row_lengths(ln, cols, seed, rng_cols)


@pytest.mark.parametrize("kind,rows,cols", CASES)
@pytest.mark.parametrize("R", [32, 64, 128])
def test_long_rows_against_the_oracle(kind, rows, cols, R, force_long_rows):
    force_long_rows()
    c, v = build(kind, rows, cols, 11)
    dims = (rows, cols)
    B = synth.random_dense((cols, R), 5).numpy()
    want, norm = oracle.spmm(c, v, dims, B)
    A = upload_packed(oracle.pack(c, v, dims, (0, 1), (D, CU)))
    C = torch.full((rows, R), float("nan"), dtype=torch.float64, device="cuda")    # every entry must be written
    before = A.handle.kernel_launches()
    comet.spmm(A, dev(B), C)
    # three analysis kernels, the two-role gather kernel, the two-role fix-up launch: the path really ran
    assert A.handle.kernel_launches() - before == 5
    assert_close(C, want, norm, what=f"spmm long rows {kind} R={R}")
    C2 = torch.full((rows, R), float("nan"), dtype=torch.float64, device="cuda")
    comet.spmm(A, dev(B), C2)
    assert torch.equal(C, C2), "the long-row path must be bit-reproducible from run to run"


@pytest.mark.parametrize("threshold,tile,piece,blocks,ctas,tile_items", [
    (40, 32, 8, 2, 1, 8), (64, 64, 16, 8, 5, 37), (40, 32, 4, 32, 2, 24), (100, 128, 64, 16, 300, 37)])
def test_long_rows_tilings(threshold, tile, piece, blocks, ctas, tile_items, force_long_rows):
    force_long_rows(threshold, tile, piece, blocks, ctas, tile_items)
    rows, cols, R = 400, 640, 64
    c, v = build("mixed", rows, cols, 12)
    B = synth.random_dense((cols, R), 6).numpy()
    want, norm = oracle.spmm(c, v, (rows, cols), B)
    A = upload_packed(oracle.pack(c, v, (rows, cols), (0, 1), (D, CU)))
    C = torch.full((rows, R), float("nan"), dtype=torch.float64, device="cuda")
    comet.spmm(A, dev(B), C)
    assert_close(C, want, norm, what="spmm long rows, tilings")


def test_long_rows_exact_small_integers(force_long_rows):
    """Small-integer values and operand: every partial sum is exact, so any order of summation must give the
    oracle's numbers bit for bit (isolates indexing from rounding)."""
    force_long_rows()
    rows, cols, R = 400, 640, 64
    c, _ = build("mixed", rows, cols, 13)
    rng = np.random.default_rng(3)
    v = rng.integers(1, 4, c[0].size).astype(np.float64) * rng.choice([-1.0, 1.0], c[0].size)
    B = rng.integers(-3, 4, (cols, R)).astype(np.float64)
    want, _ = oracle.spmm(c, v, (rows, cols), B)
    A = upload_packed(oracle.pack(c, v, (rows, cols), (0, 1), (D, CU)))
    C = comet.spmm(A, dev(B))
    assert np.array_equal(C.cpu().numpy(), want)


def test_long_rows_fp32(force_long_rows):
    force_long_rows()
    rows, cols = 400, 640
    c, v = build("mixed", rows, cols, 14)
    v32 = v.astype(np.float32)
    for R in (64, 128, 256):
        B32 = synth.random_dense((cols, R), 7).numpy().astype(np.float32)
        want, norm = oracle.spmm(c, v32.astype(np.float64), (rows, cols), B32.astype(np.float64))
        pk = oracle.pack(c, v32.astype(np.float64), (rows, cols), (0, 1), (D, CU))
        A = comet.SpTensor.from_arrays(pk.dims, pk.mode_order, pk.attr,
                                       [dev(p, torch.int32) if p.size else None for p in pk.pos],
                                       [dev(x, torch.int32) if x.size else None for x in pk.crd],
                                       dev(pk.val, torch.float32))
        C = torch.full((rows, R), float("nan"), dtype=torch.float32, device="cuda")
        comet.spmm(A, dev(B32), C)
        assert_close(C.double(), want, norm, tol=1e-5, what=f"spmm long rows fp32 R={R}")
        assert_close(C.double(), want, norm, tol=3 * 2.0 ** -24, what=f"spmm long rows fp32 R={R} (rounding bound)")


def test_scaled_workload_with_long_rows(force_long_rows):
    """The benchmark's row-length law at 1/64 scale (rows of up to ~10,000 entries next to millions of short ones)."""
    force_long_rows(threshold=128, tile=128, piece=32, blocks=8, ctas=222, tile_items=128)
    case = synth.make(2, scale=1 / 64)
    c = [x.numpy() for x in case.coords]
    v = case.val.numpy()
    B = case.dense["B"].numpy()
    want, norm = oracle.spmm(c, v, case.dims, B)
    h = comet.Handle()
    A = comet.pack([x.cuda() for x in case.coords], case.val.cuda(), case.dims, (0, 1), (D, CU), h)
    C = torch.full((case.dims[0], case.R), float("nan"), dtype=torch.float64, device="cuda")
    comet.spmm(A, dev(B), C)
    assert_close(C, want, norm, what="spmm long rows, scaled workload")


@pytest.mark.parametrize("tile_items", [16, 64, 100])
@pytest.mark.parametrize("R", [2, 16, 40])
def test_rows_around_the_length_that_one_tile_takes_whole(tile_items, R, monkeypatch):
    """Without the long-row role, a row of at most a quarter tile is processed whole by the tile that holds its
    end marker and longer rows are split with carries: rows of exactly that length, one less, one more, a whole
    tile and more, with runs of empty rows between them and at both ends of the matrix."""
    monkeypatch.setenv("COMET_SPMM_LONG_ROWS", "0")
    monkeypatch.setenv("COMET_TILE_ITEMS", str(tile_items))
    q = tile_items // 4
    rng = np.random.default_rng(tile_items + R)
    ln = []
    for _ in range(40):
        ln += [q - 1, 0, q, q + 1, 0, 0, int(rng.integers(0, q + 3)), tile_items, 1, 2 * tile_items + 3, 0, int(rng.integers(1, 4))]
    ln = [0, 0] + [max(0, x) for x in ln] + [0, q, 0]
    cols = 3 * tile_items + 50
    c, v = matrix_from_row_lengths(np.array(ln), cols, 5)
    dims = (len(ln), cols)
    B = synth.random_dense((cols, R), 8).numpy()
    want, norm = oracle.spmm(c, v, dims, B)
    A = upload_packed(oracle.pack(c, v, dims, (0, 1), (D, CU)))
    C = torch.full((dims[0], R), float("nan"), dtype=torch.float64, device="cuda")
    comet.spmm(A, dev(B), C)
    assert_close(C, want, norm, what=f"spmm tile {tile_items} R={R}")
    x = B[:, 0].copy()
    y = torch.full((dims[0],), float("nan"), dtype=torch.float64, device="cuda")
    comet.spmv(A, dev(x), y)
    wy, ny = oracle.spmv(c, v, dims, x)
    assert_close(y, wy, ny, what=f"spmv tile {tile_items}")

