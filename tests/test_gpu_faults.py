"""Host-made failures (no GPU fault is ever provoked): an allocator that refuses its n-th request must turn
every entry point into a clean COMET_ERR_ALLOC, leave nothing owned behind, and leave the handle usable."""
import ctypes as C

import numpy as np
import pytest
import torch

import oracle
import synth
from oracle import D, CU, CN, S

pytestmark = pytest.mark.gpu

comet = pytest.importorskip("paper_2102_05187_b200")
from paper_2102_05187_b200 import binding  # noqa: E402
from gpu_util import assert_close, upload_packed  # noqa: E402


class FailingHandle(comet.Handle):
    """A handle whose allocator returns NULL on request number `fail_at` (0-based), counting from arm()."""

    def __init__(self):
        super().__init__()
        self.fail_at = None
        self.calls = 0
        inner_alloc = self._alloc_cb

        def _alloc(ctx, nbytes, stream):
            n = self.calls
            self.calls += 1
            if self.fail_at is not None and n == self.fail_at:
                return None
            return inner_alloc(ctx, nbytes, stream)

        self._alloc_cb2 = binding._ALLOC_FN(_alloc)
        # a second library handle that uses the failing allocator
        self._allocator2 = binding.AllocatorStruct(self._alloc_cb2, self._free_cb, None)
        self.lib.comet_destroy(self._h)
        self._h = C.c_void_p()
        st = self.lib.comet_create(C.byref(self._h), C.byref(self._allocator2))
        assert st == 0

    def arm(self, fail_at):
        self.fail_at, self.calls = fail_at, 0


@pytest.fixture(autouse=True)
def _need_gpu(cuda_device):
    yield


def test_pack_survives_every_allocation_failure():
    h = FailingHandle()
    coords, val = synth.random_coo((60, 50, 40), 5000, 3)
    dev = [c.cuda() for c in coords]
    v = val.cuda()
    h.arm(None)
    ok = comet.pack(dev, v, (60, 50, 40), (0, 1, 2), (CU, CU, CU), h)
    total = h.calls                                   # allocations of a successful pack
    ok.free()
    assert total >= 8
    for k in range(total):
        h.arm(k)
        live_before = len(h._live)
        with pytest.raises(comet.CometError) as e:
            comet.pack(dev, v, (60, 50, 40), (0, 1, 2), (CU, CU, CU), h)
        assert e.value.status == -6
        torch.cuda.synchronize()
        assert len(h._live) == live_before, f"allocation {k}: blocks leaked"
    h.arm(None)
    again = comet.pack(dev, v, (60, 50, 40), (0, 1, 2), (CU, CU, CU), h)
    want = oracle.pack([c.numpy() for c in coords], val.numpy(), (60, 50, 40), (0, 1, 2), (CU, CU, CU))
    assert np.array_equal(again.crd(2).cpu().numpy(), want.crd[2])


def test_contractions_report_scratch_allocation_failure():
    h = FailingHandle()
    case = synth.make(2, scale=1 / 256)
    c, v = [x.numpy() for x in case.coords], case.val.numpy()
    pk = oracle.pack(c, v, case.dims, (0, 1), (D, CU))
    A = upload_packed(pk)
    A.handle = h                                       # route the calls through the failing handle
    B = case.dense["B"].cuda()
    h.arm(0)                                           # the first thing a contraction asks for is its scratch
    with pytest.raises(comet.CometError) as e:
        comet.spmm(A, B)
    assert e.value.status == -6
    h.arm(None)
    want, norm = oracle.spmm(c, v, case.dims, case.dense["B"].numpy())
    assert_close(comet.spmm(A, B), want, norm, what="spmm after a failed call")
    # symbolic outputs: every allocation of ttm_symbolic may fail
    t = synth.make(4, scale=1 / 256)
    X = comet.pack([x.cuda() for x in t.coords], t.val.cuda(), t.dims, (0, 1, 2), (CU, CU, CU), h)
    h.arm(None)
    Y = comet.ttm_symbolic(X, 2, 16)
    n_alloc = h.calls
    Y.free()
    for k in range(n_alloc):
        h.arm(k)
        live_before = len(h._live)
        with pytest.raises(comet.CometError) as e:
            comet.ttm_symbolic(X, 2, 16)
        assert e.value.status == -6 and len(h._live) == live_before


def test_sizes_beyond_the_index_types_are_refused_before_any_launch():
    """int32 indices: extents and entry counts of 2^31 - 1 or more, key widths beyond 63 bits and leading
    dimensions of 2^28 or more are reported as such; nothing is launched (the launch counter does not move)."""
    import ctypes as C
    h = comet.default_handle()
    before = h.kernel_launches()
    one = torch.zeros(1, dtype=torch.int32, device="cuda")
    v = torch.ones(1, dtype=torch.float64, device="cuda")
    for dims, status in [((1 << 31, 4), "COMET_ERR_INDEX_OVERFLOW"), ((4, (1 << 31) - 1), "COMET_ERR_INDEX_OVERFLOW"),
                         ((1 << 30, 1 << 30, 1 << 30), "COMET_ERR_UNSUPPORTED_FORMAT")]:
        with pytest.raises(comet.CometError) as e:
            comet.pack([one] * len(dims), v, dims, tuple(range(len(dims))), (comet.CU,) * len(dims))
        assert comet.binding.STATUS_NAMES[e.value.status] == status
    # a descriptor that claims more entries than int32 positions can address
    A = comet.SpTensor.from_arrays((2, 2), (0, 1), (comet.D, comet.CU),
                                   [torch.tensor([2], dtype=torch.int32, device="cuda"),
                                    torch.tensor([0, 1, 1], dtype=torch.int32, device="cuda")],
                                   [None, torch.zeros(1, dtype=torch.int32, device="cuda")], v)
    A.c.nnz = (1 << 31) + 5
    with pytest.raises(comet.CometError) as e:
        comet.spmv(A, torch.ones(2, dtype=torch.float64, device="cuda"))
    assert comet.binding.STATUS_NAMES[e.value.status] == "COMET_ERR_INDEX_OVERFLOW"
    A.c.nnz = 1
    # leading dimension of a gathered operand beyond what 32-bit byte offsets can form
    out = torch.empty((2, 1), dtype=torch.float64, device="cuda")
    st = h.lib.comet_spmm(h._h, C.byref(A.c), C.c_void_p(v.data_ptr()), C.c_int64(1), C.c_int64(1 << 28),
                          C.c_void_p(out.data_ptr()), C.c_int64(1), None)
    assert comet.binding.STATUS_NAMES[st] == "COMET_ERR_INDEX_OVERFLOW"
    assert h.kernel_launches() == before
