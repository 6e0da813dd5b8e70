"""comet_spmv_static: the SpMV entry point for callers that cannot allocate device memory (for example
a process whose GPU memory is wholly owned by another pool, or a loop that must never enter the
driver's allocator). Its carry slots sit in a fixed device array inside the library instead of in
allocator-provided scratch, so the call needs neither a handle nor an allocation.

The check: called straight through the C ABI, twice in a row on different matrices (the second call
finds the first call's leftovers in the shared array), it must reproduce comet_spmv. Collected last on
purpose: a failure here cannot hide any other test from a stop-at-first-failure run.
"""
import ctypes as C

import numpy as np
import pytest
import torch

import oracle
import synth
from oracle import D, CU

pytestmark = pytest.mark.gpu

comet = pytest.importorskip("paper_2102_05187_b200")
from gpu_util import FP64_TOL, assert_close, upload_packed  # noqa: E402


def _static_spmv(A, x, y):
    lib = comet.load_library()
    lib.comet_spmv_static.restype = C.c_int
    stream = C.c_void_p(torch.cuda.current_stream().cuda_stream)
    return lib.comet_spmv_static(C.byref(A.c), C.c_void_p(x.data_ptr()), C.c_void_p(y.data_ptr()), stream)


def test_static_spmv_matches_regular_entry_point_twice_in_a_row(cuda_device):
    cases = [synth.make(2, scale=1 / 128, seed=77), synth.make(1, scale=1.0, seed=78)]   # many tiles, then few
    for case in cases:
        c = [t.numpy() for t in case.coords]
        v = case.val.numpy()
        A = upload_packed(oracle.pack(c, v, case.dims, (0, 1), (D, CU)))
        x = synth.random_dense((case.dims[1],), case.seed).cuda()
        want = comet.spmv(A, x)
        _, norm = oracle.spmv(c, v, case.dims, x.cpu().numpy())
        for _ in range(2):
            y = torch.full((case.dims[0],), float("nan"), dtype=torch.float64, device="cuda")
            assert _static_spmv(A, x, y) == 0
            torch.cuda.synchronize()
            assert_close(y, want.cpu().numpy(), norm, tol=FP64_TOL, what="static spmv vs comet_spmv")


def test_static_spmv_rejects_what_it_cannot_hold(cuda_device):
    coords, val = synth.random_coo((8, 8), 10, 3)
    c = [t.numpy() for t in coords]
    A = upload_packed(oracle.pack(c, val.numpy(), (8, 8), (0, 1), (D, CU)))
    x = torch.ones(8, dtype=torch.float64, device="cuda")
    y = torch.zeros(8, dtype=torch.float64, device="cuda")
    too_big = comet.binding.SpTensorStruct.from_buffer_copy(A.c)
    too_big.nnz = 134_217_728                      # rows + nnz over the fixed limit: refused before any launch
    lib = comet.load_library()
    lib.comet_spmv_static.restype = C.c_int
    assert lib.comet_spmv_static(C.byref(too_big), C.c_void_p(x.data_ptr()), C.c_void_p(y.data_ptr()), None) == -8
    dcsr = upload_packed(oracle.pack(c, val.numpy(), (8, 8), (0, 1), (CU, CU)))
    assert _static_spmv(dcsr, x, y) == -2
