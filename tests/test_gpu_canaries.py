"""Stray writes: every output of the library is placed inside a larger buffer with known values on both sides, and
those values must be unchanged afterwards. Parity with the oracle cannot see a store that lands next to the output
(the kernels keep several loads and stores in flight ahead of the walk), so this is checked separately, on inputs
whose segments straddle many tiles and on every output-producing entry point."""
import numpy as np
import pytest
import torch

import oracle
import synth
from oracle import D, CU, CN, S

pytestmark = pytest.mark.gpu

comet = pytest.importorskip("paper_2102_05187_b200")
from gpu_util import assert_close, dev, upload_packed  # noqa: E402

GUARD = 4096          # elements on each side
MARK = -777.25


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


class Guarded:
    """A (rows x cols) output with leading dimension ld inside a marked buffer."""

    def __init__(self, rows, cols, ld=None, dtype=torch.float64):
        self.rows, self.cols, self.ld = rows, cols, ld or cols
        self.buf = torch.full((2 * GUARD + max(rows, 1) * self.ld,), MARK, dtype=dtype, device="cuda")
        self.view = self.buf[GUARD:GUARD + rows * self.ld].view(rows, self.ld)[:, :cols] if rows else self.buf[GUARD:GUARD]

    def check(self, what):
        assert bool((self.buf[:GUARD] == MARK).all()), f"{what}: wrote in front of the output"
        assert bool((self.buf[GUARD + self.rows * self.ld:] == MARK).all()), f"{what}: wrote behind the output"
        if self.ld > self.cols and self.rows:
            pad = self.buf[GUARD:GUARD + self.rows * self.ld].view(self.rows, self.ld)[:, self.cols:]
            assert bool((pad == MARK).all()), f"{what}: wrote into the padding between rows"


def _np(coords):
    return [c.numpy() for c in coords]


@pytest.mark.parametrize("attr", [(D, CU), (CU, CU), (CN, S)])
def test_matrix_outputs_stay_inside(attr, tile_items):
    dims = (300, 200)
    coords, val = synth.random_coo(dims, 5000, 2)
    c, v = _np(coords), val.numpy()
    A = upload_packed(oracle.pack(c, v, dims, (0, 1), attr))
    y = Guarded(dims[0], 1)
    comet.spmv(A, dev(synth.random_dense((dims[1],), 2).numpy()), y.view.reshape(-1))
    y.check("spmv")
    for R, ld in [(1, 1), (16, 16), (17, 19), (64, 64), (100, 104), (130, 130)]:
        C = Guarded(dims[0], R, ld)
        comet.spmm(A, dev(synth.random_dense((dims[1], R), 2).numpy()), C.view)
        C.check(f"spmm R={R}")
        want, norm = oracle.spmm(c, v, dims, synth.random_dense((dims[1], R), 2).numpy())
        assert_close(C.view, want, norm, what=f"spmm R={R} inside a guarded buffer")


@pytest.mark.parametrize("attr", [(CU, CU, CU), (CN, S, S)])
def test_tensor_outputs_stay_inside(attr, tile_items):
    dims = (20, 18, 16)
    coords, val = synth.random_coo(dims, 2500, 3)
    c, v = _np(coords), val.numpy()
    X = upload_packed(oracle.pack(c, v, dims, (0, 1, 2), attr))
    for R in (1, 8, 32, 40):
        out = Guarded(dims[0], R)
        F = [None, dev(synth.random_dense((dims[1], R), 3, 61).numpy()), dev(synth.random_dense((dims[2], R), 3, 62).numpy())]
        comet.mttkrp(X, 0, F, out.view)
        out.check(f"mttkrp {attr} R={R}")
        for mode in (1, 2):
            om = Guarded(dims[mode], R)
            Fm = [dev(synth.random_dense((d, R), 3, 70 + m).numpy()) for m, d in enumerate(dims)]
            Fm[mode] = None
            comet.mttkrp(X, mode, Fm, om.view)
            om.check(f"mttkrp mode {mode} {attr} R={R}")


def test_long_row_spmm_stays_inside(monkeypatch):
    for k, v in {"COMET_SPMM_LONG_MIN_NNZ": "1", "COMET_SPMM_LONG_MIN_B_MB": "0", "COMET_SPMM_LONG_ROW": "40",
                 "COMET_SPMM_LONG_TILE": "32", "COMET_SPMM_PIECE": "8", "COMET_SPMM_BLOCKS": "4", "COMET_SPMM_LONG_CTAS": "3",
                 "COMET_TILE_ITEMS": "37"}.items():
        monkeypatch.setenv(k, v)
    rng = np.random.default_rng(5)
    rows, cols, R = 200, 640, 64
    lengths = rng.integers(0, 6, rows)
    lengths[[0, 50, 51, rows - 1]] = [300, 500, 90, 250]
    ri = np.repeat(np.arange(rows), lengths).astype(np.int32)
    ci = np.concatenate([rng.choice(cols, n, replace=False) for n in lengths]).astype(np.int32)
    v = rng.uniform(-1, 1, ri.size)
    A = upload_packed(oracle.pack([ri, ci], v, (rows, cols), (0, 1), (D, CU)))
    B = synth.random_dense((cols, R), 5).numpy()
    C = Guarded(rows, R, R + 8)
    comet.spmm(A, dev(B), C.view)
    C.check("spmm, long-row path")
    want, norm = oracle.spmm([ri, ci], v, (rows, cols), B)
    assert_close(C.view, want, norm, what="spmm long rows inside a guarded buffer")
