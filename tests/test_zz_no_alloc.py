"""comet_spmv_static: the SpMV entry point for callers that cannot allocate device memory (for example
a process whose GPU memory is wholly owned by another pool, or a loop that must never enter the
driver's allocator). Its carry slots sit in a fixed device array inside the library instead of in
allocator-provided scratch, so the call needs neither a handle nor an allocation.

The check: called straight through the C ABI, twice in a row on different matrices (the second call
finds the first call's leftovers in the shared array), it must reproduce the CPU oracle's values and agree with
comet_spmv; a call must leave the amount of device memory in use unchanged; matrices without entries, with a
single tile and with trailing empty rows are covered, and so is the edge of the size limit. Collected last on
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
        regular = comet.spmv(A, x)
        want, norm = oracle.spmv(c, v, case.dims, x.cpu().numpy())
        for _ in range(2):
            y = torch.full((case.dims[0],), float("nan"), dtype=torch.float64, device="cuda")
            assert _static_spmv(A, x, y) == 0
            torch.cuda.synchronize()
            assert_close(y, want, norm, tol=FP64_TOL, what="static spmv vs the oracle")
            assert_close(y, regular.cpu().numpy(), 2 * norm, tol=FP64_TOL, what="static spmv vs comet_spmv")


def test_static_spmv_obtains_no_device_memory(cuda_device):
    """What the entry point exists for: after one warm call (which resolves the array's address), a call must not
    change the device memory in use, neither through torch's allocator nor through the driver."""
    case = synth.make(2, scale=1 / 128, seed=79)
    c = [t.numpy() for t in case.coords]
    A = upload_packed(oracle.pack(c, case.val.numpy(), case.dims, (0, 1), (D, CU)))
    x = synth.random_dense((case.dims[1],), case.seed).cuda()
    y = torch.empty(case.dims[0], dtype=torch.float64, device="cuda")
    assert _static_spmv(A, x, y) == 0
    torch.cuda.synchronize()
    free_before, _ = torch.cuda.mem_get_info()
    allocs_before = torch.cuda.memory_stats()["allocation.all.allocated"]
    assert _static_spmv(A, x, y) == 0
    torch.cuda.synchronize()
    free_after, _ = torch.cuda.mem_get_info()
    assert torch.cuda.memory_stats()["allocation.all.allocated"] == allocs_before
    assert free_after == free_before


@pytest.mark.parametrize("dims,entries", [((50, 40), []), ((7, 9), [(3, 4, 2.5)]), ((3000, 16), [(0, 1, 1.0), (0, 15, -2.0), (5, 3, 4.0)])])
def test_static_spmv_edge_shapes(cuda_device, dims, entries):
    """No entry at all (every y must become +0), one entry (a single tile), and a long tail of empty rows."""
    ci = np.array([e[0] for e in entries], dtype=np.int32)
    cj = np.array([e[1] for e in entries], dtype=np.int32)
    v = np.array([e[2] for e in entries], dtype=np.float64)
    A = upload_packed(oracle.pack([ci, cj], v, dims, (0, 1), (D, CU)))
    xh = np.arange(1, dims[1] + 1, dtype=np.float64)
    want, norm = oracle.spmv([ci, cj], v, dims, xh)
    y = torch.full((dims[0],), float("nan"), dtype=torch.float64, device="cuda")
    assert _static_spmv(A, torch.from_numpy(xh).cuda(), y) == 0
    torch.cuda.synchronize()
    assert_close(y, want, norm, tol=FP64_TOL, what="static spmv, edge shape")
    assert not torch.signbit(y[torch.from_numpy(norm == 0).cuda()]).any()


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
    # rows + nnz exactly at the limit is legal: the size check lets it through, and the next check (a NULL value
    # array) stops the call before anything is launched on the made-up sizes
    at_limit = comet.binding.SpTensorStruct.from_buffer_copy(A.c)
    at_limit.nnz = 134_217_728 - 8
    at_limit.val = None
    assert lib.comet_spmv_static(C.byref(at_limit), C.c_void_p(x.data_ptr()), C.c_void_p(y.data_ptr()), None) == -1
    dcsr = upload_packed(oracle.pack(c, val.numpy(), (8, 8), (0, 1), (CU, CU)))
    assert _static_spmv(dcsr, x, y) == -2
