"""Thin ctypes binding of libcomet.so (include/comet.h): argument marshalling only.

PyTorch is used for device memory and streams: operands are torch CUDA tensors whose `data_ptr()` is
passed through, the library allocates its data-dependent outputs through a callback that hands out
torch tensors (so they live in torch's caching allocator), and every call runs on torch's current
stream. Every step of the contractions and of the packing runs in the library's CUDA kernels; there is
no fallback: importing this module without a built libcomet.so, or calling it without a GPU, raises.
"""
from __future__ import annotations

import ctypes as C
import os

import torch

D, CU, CN, S = 0, 1, 2, 3
F64 = 0
F32 = 1
_TORCH_DTYPE = {F64: torch.float64, F32: torch.float32}


def _dtype_code(t: torch.Tensor) -> int:
    """comet_dtype_t of a value tensor (fp64 or fp32; anything else is refused here)."""
    if t.dtype == torch.float64:
        return F64
    if t.dtype == torch.float32:
        return F32
    raise TypeError(f"values must be float64 or float32, got {t.dtype}")


def _same_dtype(A, *tensors):
    want = _TORCH_DTYPE[A.c.dtype]
    for t in tensors:
        if t is not None and t.dtype != want:
            raise TypeError(f"dense operand is {t.dtype}, the sparse tensor's values are {want}")
    return want
MAX_ORDER = 4

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libcomet.so")

STATUS_NAMES = {
    0: "COMET_OK", -1: "COMET_ERR_INVALID_ARG", -2: "COMET_ERR_UNSUPPORTED_FORMAT",
    -3: "COMET_ERR_COORD_OUT_OF_RANGE", -4: "COMET_ERR_DUPLICATE_COORD", -5: "COMET_ERR_INDEX_OVERFLOW",
    -6: "COMET_ERR_ALLOC", -7: "COMET_ERR_CUDA", -8: "COMET_ERR_WORKSPACE", -9: "COMET_ERR_MISALIGNED",
    -10: "COMET_ERR_INVALID_TENSOR",
}

EXPORTS = [
    "comet_create", "comet_destroy", "comet_status_string", "comet_last_cuda_error", "comet_kernel_launches",
    "comet_pack",
    "comet_sptensor_free", "comet_validate", "comet_spmv", "comet_spmm", "comet_ttv_symbolic", "comet_ttv",
    "comet_ttm_symbolic", "comet_ttm", "comet_mttkrp", "comet_spmv_static", "comet_pack_ex", "comet_ttm_symbolic_ex", "comet_reorder",
    "comet_elementwise_mul", "comet_spmm_from_host",
]


class CometError(RuntimeError):
    def __init__(self, status: int, what: str, detail: str = ""):
        name = STATUS_NAMES.get(status, str(status))
        super().__init__(f"{what}: {name}{(' (' + detail + ')') if detail else ''}")
        self.status = status


class SpTensorStruct(C.Structure):
    _fields_ = [
        ("order", C.c_int32), ("dtype", C.c_int32),
        ("dims", C.c_int64 * MAX_ORDER),
        ("mode_order", C.c_int32 * MAX_ORDER),
        ("attr", C.c_int32 * MAX_ORDER),
        ("pos", C.c_void_p * MAX_ORDER), ("pos_len", C.c_int64 * MAX_ORDER),
        ("crd", C.c_void_p * MAX_ORDER), ("crd_len", C.c_int64 * MAX_ORDER),
        ("val", C.c_void_p), ("nnz", C.c_int64),
        ("owner", C.c_void_p),
    ]


_ALLOC_FN = C.CFUNCTYPE(C.c_void_p, C.c_void_p, C.c_size_t, C.c_void_p)
_FREE_FN = C.CFUNCTYPE(None, C.c_void_p, C.c_void_p, C.c_void_p)


class AllocatorStruct(C.Structure):
    _fields_ = [("alloc", _ALLOC_FN), ("free", _FREE_FN), ("ctx", C.c_void_p)]


_lib = None


def load_library():
    """Loads libcomet.so; raises if it has not been built (python -m paper_2102_05187_b200.build)."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise ImportError(f"{LIB_PATH} is missing: build it with `python -m paper_2102_05187_b200.build` "
                          "(there is no fallback path)")
    lib = C.CDLL(LIB_PATH)
    for name in EXPORTS:
        if not hasattr(lib, name):
            raise ImportError(f"libcomet.so does not export {name}")
    lib.comet_status_string.restype = C.c_char_p
    lib.comet_status_string.argtypes = [C.c_int]
    lib.comet_kernel_launches.restype = C.c_int64
    lib.comet_kernel_launches.argtypes = [C.c_void_p]
    for name in EXPORTS:
        if name not in ("comet_status_string", "comet_kernel_launches"):
            getattr(lib, name).restype = C.c_int
    _lib = lib
    return lib


def _stream_ptr():
    return C.c_void_p(torch.cuda.current_stream().cuda_stream)


def _ptr(t):
    return C.c_void_p(0 if t is None else t.data_ptr())


def _require_cuda(*tensors):
    for t in tensors:
        if t is not None and not t.is_cuda:
            raise ValueError("operands must be CUDA tensors: the library has no host path")


class Handle:
    """A library handle whose allocator hands out torch CUDA tensors."""

    def __init__(self):
        if not torch.cuda.is_available():
            raise RuntimeError("libcomet needs a CUDA device: there is no CPU fallback")
        self.lib = load_library()
        self._live = {}

        def _alloc(_ctx, nbytes, _stream):
            try:
                t = torch.empty(max(int(nbytes), 1), dtype=torch.uint8, device="cuda")
            except Exception:
                return None
            self._live[t.data_ptr()] = t
            return t.data_ptr()

        def _free(_ctx, ptr, _stream):
            self._live.pop(ptr, None)

        self._alloc_cb = _ALLOC_FN(_alloc)
        self._free_cb = _FREE_FN(_free)
        self._allocator = AllocatorStruct(self._alloc_cb, self._free_cb, None)
        self._h = C.c_void_p()
        st = self.lib.comet_create(C.byref(self._h), C.byref(self._allocator))
        if st:
            raise CometError(st, "comet_create")

    def close(self):
        if getattr(self, "_h", None) is not None and self._h:
            self.lib.comet_destroy(self._h)
            self._h = C.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def kernel_launches(self) -> int:
        """Kernels launched through this handle so far."""
        return int(self.lib.comet_kernel_launches(self._h))

    def check(self, st: int, what: str):
        if st:
            detail = ""
            if st == -7:
                detail = f"cudaError {self.lib.comet_last_cuda_error(self._h)}"
            raise CometError(st, what, detail)


_default_handle = None


def default_handle() -> Handle:
    global _default_handle
    if _default_handle is None:
        _default_handle = Handle()
    return _default_handle


class SpTensor:
    """A sparse tensor descriptor plus whatever keeps its device arrays alive.

    Library-owned tensors (from pack / *_symbolic) are released on `free()` or garbage collection;
    caller-built ones (from `from_arrays`) borrow the torch tensors they were given.
    """

    def __init__(self, handle: Handle, struct: SpTensorStruct, keep=None):
        self.handle = handle
        self.c = struct
        self._keep = keep

    @property
    def order(self):
        return self.c.order

    @property
    def nnz(self):
        return self.c.nnz

    @property
    def dims(self):
        return tuple(self.c.dims[m] for m in range(self.c.order))

    @property
    def attr(self):
        return tuple(self.c.attr[l] for l in range(self.c.order))

    @property
    def mode_order(self):
        return tuple(self.c.mode_order[l] for l in range(self.c.order))

    def pos(self, l):
        return _from_ptr(self.c.pos[l], self.c.pos_len[l], torch.int32, self)

    def crd(self, l):
        return _from_ptr(self.c.crd[l], self.c.crd_len[l], torch.int32, self)

    @property
    def val(self):
        return _from_ptr(self.c.val, self.c.nnz, _TORCH_DTYPE[self.c.dtype], self)

    def free(self):
        if self.c.owner:
            self.handle.lib.comet_sptensor_free(self.handle._h, C.byref(self.c), _stream_ptr())
        self._keep = None

    def __del__(self):
        try:
            self.free()
        except Exception:
            pass

    @staticmethod
    def from_arrays(dims, mode_order, attr, pos, crd, val, handle: Handle | None = None) -> "SpTensor":
        """Describe caller-built level arrays (torch CUDA int32 tensors, float64 or float32 values; None where a
        level has none)."""
        handle = handle or default_handle()
        s = SpTensorStruct()
        order = len(dims)
        s.order, s.dtype = order, _dtype_code(val)
        keep = []
        for m in range(order):
            s.dims[m] = int(dims[m])
            s.mode_order[m] = int(mode_order[m])
            s.attr[m] = int(attr[m])
            p = pos[m] if pos[m] is not None and pos[m].numel() else None
            c = crd[m] if crd[m] is not None and crd[m].numel() else None
            for t in (p, c):
                if t is not None:
                    _require_cuda(t)
                    assert t.dtype == torch.int32 and t.is_contiguous()
                    keep.append(t)
            s.pos[m] = 0 if p is None else p.data_ptr()
            s.pos_len[m] = 0 if p is None else p.numel()
            s.crd[m] = 0 if c is None else c.data_ptr()
            s.crd_len[m] = 0 if c is None else c.numel()
        _require_cuda(val)
        assert val.is_contiguous()
        keep.append(val)
        s.val = val.data_ptr() if val.numel() else 0
        s.nnz = val.numel()
        s.owner = None
        return SpTensor(handle, s, keep)


def _from_ptr(ptr, n, dtype, owner):
    """A torch tensor aliasing n elements of device memory at ptr (kept alive by `owner`)."""
    if not ptr or n == 0:
        return torch.zeros(0, dtype=dtype, device="cuda")
    itemsize = torch.empty(0, dtype=dtype).element_size()

    class _Iface:
        pass

    iface = _Iface()
    typestr = {torch.int32: "<i4", torch.float64: "<f8", torch.float32: "<f4", torch.uint8: "|u1"}[dtype]
    iface.__cuda_array_interface__ = {"shape": (int(n),), "typestr": typestr, "data": (int(ptr), False),
                                      "version": 3, "strides": (itemsize,)}
    iface._owner = owner
    return torch.as_tensor(iface, device="cuda")


# ------------------------------------------------------------------------------------------- entry points

PACK_SUM_DUPLICATES = 1
PACK_CSR_HISTOGRAM = 2


def pack(coords, val, dims, mode_order, attr, handle: Handle | None = None, sum_duplicates: bool = False,
         csr_histogram: bool = False) -> SpTensor:
    """comet_pack / comet_pack_ex: COO (one int32 CUDA tensor per mode, any order) -> packed levels. Cells must be
    distinct unless `sum_duplicates`, which merges equal cells (values added in input order). `csr_histogram`:
    for [D,CU] matrices with rows of similar length, build the rows as a histogram instead of a full sort."""
    handle = handle or default_handle()
    order = len(dims)
    _require_cuda(val, *coords)
    coords = [c.contiguous() for c in coords]
    val = val.contiguous()
    assert all(c.dtype == torch.int32 for c in coords)
    h_dims = (C.c_int64 * order)(*[int(d) for d in dims])
    h_crd = (C.c_void_p * order)(*[c.data_ptr() for c in coords])
    h_mo = (C.c_int32 * order)(*[int(m) for m in mode_order])
    h_at = (C.c_int32 * order)(*[int(a) for a in attr])
    out = SpTensorStruct()
    st = handle.lib.comet_pack_ex(handle._h, C.c_int32(order), h_dims, C.c_int64(val.numel()), h_crd, _ptr(val),
                                  C.c_int(_dtype_code(val)), h_mo, h_at,
                                  C.c_uint32((PACK_SUM_DUPLICATES if sum_duplicates else 0) | (PACK_CSR_HISTOGRAM if csr_histogram else 0)),
                                  _stream_ptr(),
                                  C.byref(out))
    handle.check(st, "comet_pack")
    return SpTensor(handle, out)


def validate(t: SpTensor):
    t.handle.check(t.handle.lib.comet_validate(t.handle._h, C.byref(t.c), _stream_ptr()), "comet_validate")


def spmv(A: SpTensor, x: torch.Tensor, y: torch.Tensor | None = None) -> torch.Tensor:
    _require_cuda(x)
    rows = A.c.dims[A.c.mode_order[0]]
    dt = _same_dtype(A, x, y)
    if y is None:
        y = torch.empty(rows, dtype=dt, device=x.device)
    st = A.handle.lib.comet_spmv(A.handle._h, C.byref(A.c), _ptr(x), _ptr(y), _stream_ptr())
    A.handle.check(st, "comet_spmv")
    return y


def spmm(A: SpTensor, B: torch.Tensor, out: torch.Tensor | None = None) -> torch.Tensor:
    _require_cuda(B)
    assert B.dim() == 2 and B.stride(1) == 1
    rows = A.c.dims[A.c.mode_order[0]]
    R = B.shape[1]
    dt = _same_dtype(A, B, out)
    if out is None:
        out = torch.empty((rows, R), dtype=dt, device=B.device)
    st = A.handle.lib.comet_spmm(A.handle._h, C.byref(A.c), _ptr(B), C.c_int64(R), C.c_int64(B.stride(0)),
                                 _ptr(out), C.c_int64(out.stride(0)), _stream_ptr())
    A.handle.check(st, "comet_spmm")
    return out


def elementwise_mul(A: SpTensor, B: torch.Tensor, out_val: torch.Tensor | None = None) -> SpTensor:
    """C = A .* B for a dense B over A's modes (any strides): a tensor that shares A's level arrays (A must
    outlive it) and owns its values."""
    _require_cuda(B)
    dt = _same_dtype(A, B, out_val)
    modes = 2 if A.attr == (D, D, S) else A.c.order
    assert B.dim() == modes
    if out_val is None:
        out_val = torch.empty(A.c.nnz, dtype=dt, device=B.device)
    strides = (C.c_int64 * MAX_ORDER)(*[int(x) for x in B.stride()], *([0] * (MAX_ORDER - modes)))
    st = A.handle.lib.comet_elementwise_mul(A.handle._h, C.byref(A.c), _ptr(B), strides, _ptr(out_val), _stream_ptr())
    A.handle.check(st, "comet_elementwise_mul")
    s = SpTensorStruct.from_buffer_copy(A.c)
    s.val = out_val.data_ptr() if out_val.numel() else 0
    s.owner = None
    return SpTensor(A.handle, s, keep=[A, out_val])


def ttv_symbolic(X: SpTensor, mode: int, out_attr=None) -> SpTensor:
    """Structure of X x_mode v: one level fewer than X. Default format: CSR [D,CU] for a 3-order X,
    CSF [CU,CU,CU] for a 4-order X."""
    out = SpTensorStruct()
    n = X.c.order - 1
    if out_attr is None:
        out_attr = (D, CU) if n == 2 else (CU,) * n
    assert len(out_attr) == n
    h_at = (C.c_int32 * n)(*out_attr)
    st = X.handle.lib.comet_ttv_symbolic(X.handle._h, C.byref(X.c), C.c_int32(mode), h_at, _stream_ptr(), C.byref(out))
    X.handle.check(st, "comet_ttv_symbolic")
    return SpTensor(X.handle, out)


def ttv(X: SpTensor, mode: int, v: torch.Tensor, Y: SpTensor | None = None) -> SpTensor:
    _require_cuda(v)
    _same_dtype(X, v)
    if Y is None:
        Y = ttv_symbolic(X, mode)
    st = X.handle.lib.comet_ttv(X.handle._h, C.byref(X.c), C.c_int32(mode), _ptr(v), C.byref(Y.c), _stream_ptr())
    X.handle.check(st, "comet_ttv")
    return Y


def ttm_symbolic(X: SpTensor, mode: int, R: int, out_attr=None) -> SpTensor:
    """Structure of X x_mode U. out_attr: None (compressed levels + dense last level) or, for a 3-order X,
    (CN, S, D): the mode-generic form with one coordinate pair per stored fiber."""
    out = SpTensorStruct()
    h_at = None if out_attr is None else (C.c_int32 * X.c.order)(*out_attr)
    st = X.handle.lib.comet_ttm_symbolic_ex(X.handle._h, C.byref(X.c), C.c_int32(mode), C.c_int64(R), h_at,
                                            _stream_ptr(), C.byref(out))
    X.handle.check(st, "comet_ttm_symbolic")
    return SpTensor(X.handle, out)


def ttm(X: SpTensor, mode: int, U: torch.Tensor, Y: SpTensor | None = None) -> SpTensor:
    _require_cuda(U)
    assert U.dim() == 2 and U.stride(1) == 1
    R = U.shape[1]
    _same_dtype(X, U)
    if Y is None:
        Y = ttm_symbolic(X, mode, R)
    st = X.handle.lib.comet_ttm(X.handle._h, C.byref(X.c), C.c_int32(mode), _ptr(U), C.c_int64(R),
                                C.c_int64(U.stride(0)), C.byref(Y.c), _stream_ptr())
    X.handle.check(st, "comet_ttm")
    return Y


def mttkrp(X: SpTensor, mode: int, factors, out: torch.Tensor | None = None) -> torch.Tensor:
    """factors: one (dims[m] x R) CUDA tensor per mode; the entry at `mode` may be None."""
    live = [f for m, f in enumerate(factors) if m != mode and f is not None]
    _require_cuda(*live)
    R = live[0].shape[1]
    assert all(f.dim() == 2 and f.stride(1) == 1 and f.shape[1] == R for f in live)
    rows = X.c.dims[mode]
    dt = _same_dtype(X, out, *live)
    if out is None:
        out = torch.empty((rows, R), dtype=dt, device=live[0].device)
    order = X.c.order
    assert len(factors) == order
    h_f = (C.c_void_p * order)(*[0 if (m == mode or f is None) else f.data_ptr() for m, f in enumerate(factors)])
    h_ld = (C.c_int64 * order)(*[0 if (m == mode or f is None) else f.stride(0) for m, f in enumerate(factors)])
    st = X.handle.lib.comet_mttkrp(X.handle._h, C.byref(X.c), C.c_int32(mode), h_f, h_ld, C.c_int64(R), _ptr(out),
                                   C.c_int64(out.stride(0)), _stream_ptr())
    X.handle.check(st, "comet_mttkrp")
    return out


def reorder(coords, dims, iterations: int = 5, handle: Handle | None = None):
    """comet_reorder: new numbers for the indices of every mode (one int32 CUDA tensor per mode) that gather
    the entries around the diagonal. Apply with `label[m][coords[m].long()]`; dense operands and results
    indexed by mode m move their rows accordingly."""
    handle = handle or default_handle()
    order = len(dims)
    _require_cuda(*coords)
    coords = [c.contiguous() for c in coords]
    assert all(c.dtype == torch.int32 for c in coords)
    labels = [torch.empty(int(d), dtype=torch.int32, device=coords[0].device) for d in dims]
    h_dims = (C.c_int64 * order)(*[int(d) for d in dims])
    h_crd = (C.c_void_p * order)(*[c.data_ptr() for c in coords])
    h_lab = (C.c_void_p * order)(*[l.data_ptr() for l in labels])
    st = handle.lib.comet_reorder(handle._h, C.c_int32(order), h_dims, C.c_int64(coords[0].numel()), h_crd,
                                  C.c_int32(iterations), h_lab, _stream_ptr())
    handle.check(st, "comet_reorder")
    return labels


def spmm_from_host(h_coords, h_val, dims, h_B, h_out, handle: Handle | None = None):
    """comet_spmm_from_host: the whole SpMM path from HOST buffers (pinned host tensors make the copies
    asynchronous): COO entries and B in, CSR packing, multiplication, C back into `h_out`, with B and C
    travelling in column chunks so that the two directions of the bus overlap. Returns after the result has
    landed in `h_out`."""
    handle = handle or default_handle()
    tensors = list(h_coords) + [h_val, h_B, h_out]
    if any(t.is_cuda for t in tensors):
        raise ValueError("spmm_from_host takes host tensors")
    assert len(h_coords) == 2 and all(c.dtype == torch.int32 and c.is_contiguous() for c in h_coords)
    assert h_val.is_contiguous() and h_B.dim() == 2 and h_out.dim() == 2 and h_B.stride(1) == 1 and h_out.stride(1) == 1
    assert h_B.dtype == h_val.dtype == h_out.dtype
    R = int(h_B.shape[1])
    assert tuple(h_out.shape) == (int(dims[0]), R) and int(h_B.shape[0]) == int(dims[1])
    h_dims = (C.c_int64 * 2)(int(dims[0]), int(dims[1]))
    st = handle.lib.comet_spmm_from_host(handle._h, h_dims, C.c_int64(h_val.numel()), _ptr(h_coords[0]), _ptr(h_coords[1]),
                                         _ptr(h_val), C.c_int32(_dtype_code(h_val)), _ptr(h_B), C.c_int64(h_B.stride(0)),
                                         C.c_int64(R), _ptr(h_out), C.c_int64(h_out.stride(0)), _stream_ptr())
    handle.check(st, "comet_spmm_from_host")
    return h_out
