"""ctypes front end of the CPU oracle (oracle/comet_oracle.c).

TEST INFRASTRUCTURE ONLY. Nothing on the product path may import this package: it is for the tests,
the smoke check and the benchmark's CPU-baseline leg. It shares no code with the CUDA library.

All arguments are numpy arrays (or anything `numpy.asarray` accepts); coordinates are int32, values
and dense operands float64. Contractions take the RAW COO entries and return `(result, normaliser)`
where `normaliser[e] = sum |x| |b| (|c|)` over the terms of output element e; a candidate r agrees
with the oracle when `|r - result| <= tol * normaliser`.
"""
from __future__ import annotations

import ctypes as C
from dataclasses import dataclass

import numpy as np

from .build import build as _build

D, CU, CN, S = 0, 1, 2, 3
MAX_ORDER = 4

_lib = None


class OracleError(RuntimeError):
    def __init__(self, code: int, what: str):
        super().__init__(f"oracle {what} failed with code {code}")
        self.code = code


def lib():
    global _lib
    if _lib is None:
        _lib = C.CDLL(_build())
        _lib.oracle_fiber_keys.restype = C.c_int64
        _lib.oracle_fiber_keys_n.restype = C.c_int64
    return _lib


def _i32(a):
    return np.ascontiguousarray(np.asarray(a), dtype=np.int32)


def _f64(a):
    return np.ascontiguousarray(np.asarray(a), dtype=np.float64)


def _i64(a):
    return np.ascontiguousarray(np.asarray(a), dtype=np.int64)


def _p(a):
    return None if a is None else a.ctypes.data_as(C.c_void_p)


def _slots(rows, dim):
    """rows (ascending sample of output rows, or None) -> (slot map or None, number of outputs)."""
    if rows is None:
        return None, dim
    rows = _i64(rows)
    slot = np.full(dim, -1, dtype=np.int64)
    slot[rows] = np.arange(len(rows), dtype=np.int64)
    return slot, len(rows)


def spmv(coords, val, dims, x, rows=None):
    """y_i = sum_j X_ij x_j over raw COO entries. `rows`: optional subset of output rows."""
    ci, cj = _i32(coords[0]), _i32(coords[1])
    val, x = _f64(val), _f64(x)
    slot, n_out = _slots(rows, dims[0])
    y = np.zeros(n_out)
    yn = np.zeros(n_out)
    rc = lib().oracle_spmv(C.c_int64(len(val)), _p(ci), _p(cj), _p(val), C.c_int64(dims[0]), C.c_int64(dims[1]),
                           _p(x), _p(slot), C.c_int64(n_out), _p(y), _p(yn))
    if rc:
        raise OracleError(rc, "spmv")
    return y, yn


def spmm(coords, val, dims, B, rows=None):
    """Y_ir = sum_j X_ij B_jr; B row-major (J x R)."""
    ci, cj = _i32(coords[0]), _i32(coords[1])
    val, B = _f64(val), _f64(B)
    R = B.shape[1]
    slot, n_out = _slots(rows, dims[0])
    Y = np.zeros((n_out, R))
    Yn = np.zeros((n_out, R))
    rc = lib().oracle_spmm(C.c_int64(len(val)), _p(ci), _p(cj), _p(val), C.c_int64(dims[0]), C.c_int64(dims[1]),
                           _p(B), C.c_int64(R), C.c_int64(R), _p(slot), C.c_int64(n_out), _p(Y), _p(Yn))
    if rc:
        raise OracleError(rc, "spmm")
    return Y, Yn


def fiber_keys(coords, dims, mode):
    """Sorted distinct keys a*dim_b+b of the two kept modes (a<b) for a mode-`mode` TTV/TTM."""
    c = [_i32(x) for x in coords]
    keys = np.zeros(max(1, len(c[0])), dtype=np.int64)
    d = _i64(dims)
    n = lib().oracle_fiber_keys(C.c_int64(len(c[0])), _p(c[0]), _p(c[1]), _p(c[2]), _p(d), C.c_int(mode), _p(keys))
    if n < 0:
        raise OracleError(n, "fiber_keys")
    return keys[:n].copy()


def _coord_ptrs(c):
    return (C.c_void_p * len(c))(*[x.ctypes.data for x in c])


def fiber_keys_n(coords, dims, mode):
    """Sorted distinct keys of the kept modes (linearised in increasing mode order) for tensors of order 2..4."""
    c = [_i32(x) for x in coords]
    keys = np.zeros(max(1, len(c[0])), dtype=np.int64)
    n = lib().oracle_fiber_keys_n(C.c_int(len(dims)), C.c_int64(len(c[0])), _coord_ptrs(c), _p(_i64(dims)),
                                  C.c_int(mode), _p(keys))
    if n < 0:
        raise OracleError(n, "fiber_keys_n")
    return keys[:n].copy()


def ttm_n(coords, val, dims, mode, U, keys=None):
    """Y = X x_mode U for tensors of order 2..4 (U is I_mode x R; one column = tensor times vector).
    Returns (keys, Y[nkeys, R], normaliser)."""
    c = [_i32(x) for x in coords]
    val, U = _f64(val), _f64(U)
    if U.ndim == 1:
        U = U.reshape(-1, 1)
    R = U.shape[1]
    keys = fiber_keys_n(coords, dims, mode) if keys is None else _i64(keys)
    Y = np.zeros((len(keys), R))
    Yn = np.zeros((len(keys), R))
    rc = lib().oracle_ttm_n(C.c_int(len(dims)), C.c_int64(len(val)), _coord_ptrs(c), _p(val), _p(_i64(dims)),
                            C.c_int(mode), _p(U), C.c_int64(R), C.c_int64(R), _p(keys), C.c_int64(len(keys)), _p(Y),
                            _p(Yn))
    if rc:
        raise OracleError(rc, "ttm_n")
    return keys, Y, Yn


def ttv(coords, val, dims, mode, v, keys=None):
    """Y = X x_mode v. Returns (keys, values, normaliser): one value per distinct kept-coordinate pair,
    keys ascending (= lexicographic order of the kept modes)."""
    c = [_i32(x) for x in coords]
    val, v = _f64(val), _f64(v)
    d = _i64(dims)
    keys = fiber_keys(coords, dims, mode) if keys is None else _i64(keys)
    y = np.zeros(len(keys))
    yn = np.zeros(len(keys))
    rc = lib().oracle_ttv(C.c_int64(len(val)), _p(c[0]), _p(c[1]), _p(c[2]), _p(val), _p(d), C.c_int(mode), _p(v),
                          _p(keys), C.c_int64(len(keys)), _p(y), _p(yn))
    if rc:
        raise OracleError(rc, "ttv")
    return keys, y, yn


def ttm(coords, val, dims, mode, U, keys=None):
    """Y = X x_mode U with U (I_mode x R). Returns (keys, Y[nkeys, R], normaliser)."""
    c = [_i32(x) for x in coords]
    val, U = _f64(val), _f64(U)
    R = U.shape[1]
    d = _i64(dims)
    keys = fiber_keys(coords, dims, mode) if keys is None else _i64(keys)
    Y = np.zeros((len(keys), R))
    Yn = np.zeros((len(keys), R))
    rc = lib().oracle_ttm(C.c_int64(len(val)), _p(c[0]), _p(c[1]), _p(c[2]), _p(val), _p(d), C.c_int(mode), _p(U),
                          C.c_int64(R), C.c_int64(R), _p(keys), C.c_int64(len(keys)), _p(Y), _p(Yn))
    if rc:
        raise OracleError(rc, "ttm")
    return keys, Y, Yn


def mttkrp(coords, val, dims, mode, factors, rows=None):
    """out_{i_mode, r} = sum x * P_pr * Q_qr over the two other modes (increasing mode order).
    `factors`: three (dim_m x R) arrays; the one at `mode` is ignored (may be None)."""
    c = [_i32(x) for x in coords]
    val = _f64(val)
    d = _i64(dims)
    F = [None if (m == mode or f is None) else _f64(f) for m, f in enumerate(factors)]
    R = next(f.shape[1] for f in F if f is not None)
    ld = _i64([R, R, R])
    slot, n_out = _slots(rows, dims[mode])
    A = np.zeros((n_out, R))
    An = np.zeros((n_out, R))
    rc = lib().oracle_mttkrp(C.c_int64(len(val)), _p(c[0]), _p(c[1]), _p(c[2]), _p(val), _p(d), C.c_int(mode),
                             _p(F[0]), _p(F[1]), _p(F[2]), _p(ld), C.c_int64(R), _p(slot), C.c_int64(n_out),
                             _p(A), _p(An))
    if rc:
        raise OracleError(rc, "mttkrp")
    return A, An


def mttkrp_n(coords, val, dims, mode, factors, rows=None):
    """MTTKRP for tensors of order 3 or 4: out_{i_mode, r} = sum x * prod of the other modes' factor entries.
    `factors`: one (dim_m x R) array per mode; the one at `mode` is ignored (may be None)."""
    order = len(dims)
    c = [_i32(x) for x in coords]
    val = _f64(val)
    F = [None if (m == mode or f is None) else _f64(f) for m, f in enumerate(factors)]
    R = next(f.shape[1] for f in F if f is not None)
    fp = (C.c_void_p * order)(*[None if f is None else f.ctypes.data for f in F])
    slot, n_out = _slots(rows, dims[mode])
    A = np.zeros((n_out, R))
    An = np.zeros((n_out, R))
    rc = lib().oracle_mttkrp_n(C.c_int(order), C.c_int64(len(val)), _coord_ptrs(c), _p(val), _p(_i64(dims)),
                               C.c_int(mode), fp, _p(_i64([R] * order)), C.c_int64(R), _p(slot), C.c_int64(n_out),
                               _p(A), _p(An))
    if rc:
        raise OracleError(rc, "mttkrp_n")
    return A, An


class _Packed(C.Structure):
    _fields_ = [("order", C.c_int32), ("nnz", C.c_int64),
                ("pos", C.c_void_p * MAX_ORDER), ("pos_len", C.c_int64 * MAX_ORDER),
                ("crd", C.c_void_p * MAX_ORDER), ("crd_len", C.c_int64 * MAX_ORDER),
                ("val", C.c_void_p), ("perm", C.c_void_p)]


@dataclass
class Packed:
    """Per-level arrays of a packed tensor: pos[l], crd[l] (int32; empty where the attribute has none),
    val (float64, leaf order), perm (input index of the entry at each leaf position)."""
    dims: tuple
    mode_order: tuple
    attr: tuple
    pos: list
    crd: list
    val: np.ndarray
    perm: np.ndarray


def _copy(ptr, n, dtype):
    if not ptr or n == 0:
        return np.zeros(0, dtype=dtype)
    return np.ctypeslib.as_array(C.cast(ptr, C.POINTER(np.ctypeslib.as_ctypes_type(dtype))), shape=(n,)).copy()


def sum_duplicates(coords, val, dims, mode_order):
    """Merge entries with equal coordinates (values added one by one in double, in input order).
    Returns (coords, val, first): the merged entries sorted in storage order and, for each, the input
    index of its first contributor."""
    order = len(dims)
    c = [_i32(x) for x in coords]
    val = _f64(val)
    n = len(val)
    oc = [np.zeros(max(n, 1), dtype=np.int32) for _ in range(order)]
    ov = np.zeros(max(n, 1))
    first = np.zeros(max(n, 1), dtype=np.int64)
    lib().oracle_sum_duplicates.restype = C.c_int64
    m = lib().oracle_sum_duplicates(C.c_int32(order), C.c_int64(n), _coord_ptrs(c), _p(val), _p(_i32(mode_order)),
                                    _coord_ptrs(oc), _p(ov), _p(first))
    if m < 0:
        raise OracleError(m, "sum_duplicates")
    return [x[:m].copy() for x in oc], ov[:m].copy(), first[:m].copy()


def pack(coords, val, dims, mode_order, attr, sum_duplicates_first: bool = False) -> Packed:
    """COO -> level arrays for the given storage order and per-level attributes (D, CU, CN, S).
    Entries with equal coordinates are an error unless `sum_duplicates_first`, in which case they are
    merged (see sum_duplicates) before packing; `perm` then refers to the merged entry list."""
    order = len(dims)
    if sum_duplicates_first:
        coords, val, _ = sum_duplicates(coords, val, dims, mode_order)
    c = [_i32(x) for x in coords]
    val = _f64(val)
    ptrs = (C.c_void_p * order)(*[a.ctypes.data for a in c])
    d = _i64(dims)
    mo = _i32(mode_order)
    at = _i32(attr)
    out = _Packed()
    rc = lib().oracle_pack(C.c_int32(order), _p(d), C.c_int64(len(val)), ptrs, _p(val), _p(mo), _p(at), C.byref(out))
    if rc:
        raise OracleError(rc, "pack")
    try:
        n = out.nnz
        res = Packed(tuple(dims), tuple(mode_order), tuple(attr),
                     [_copy(out.pos[l], out.pos_len[l], np.int32) for l in range(order)],
                     [_copy(out.crd[l], out.crd_len[l], np.int32) for l in range(order)],
                     _copy(out.val, n, np.float64), _copy(out.perm, n, np.int64))
    finally:
        lib().oracle_packed_free(C.byref(out))
    return res
