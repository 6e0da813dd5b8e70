"""ctypes front end of oracle/timed_baseline.c: the oracle's SpMM loop with double accumulators, built
-O3 -march=native, on 1..n threads. TEST INFRASTRUCTURE ONLY (the benchmark's CPU-baseline leg and its pin)."""
from __future__ import annotations

import ctypes as C
import os
import subprocess

import numpy as np

HERE = os.path.dirname(os.path.abspath(__file__))
SRC = os.path.join(HERE, "timed_baseline.c")
LIB = os.path.join(HERE, "libcomet_timed_baseline.so")
_lib = None


def build(force: bool = False) -> str:
    if not force and os.path.exists(LIB) and os.path.getmtime(LIB) >= os.path.getmtime(SRC):
        return LIB
    subprocess.run(["gcc", "-O3", "-march=native", "-std=c11", "-fPIC", "-shared", "-pthread", "-Wall", "-Wextra",
                    "-o", LIB, SRC], check=True)
    return LIB


def host_threads() -> int:
    """Threads this process may run on (the scheduler affinity mask, not the machine's core count)."""
    return len(os.sched_getaffinity(0))


def spmm(coords, val, dims, B, threads: int = 1) -> np.ndarray:
    global _lib
    if _lib is None:
        _lib = C.CDLL(build())
    ci = np.ascontiguousarray(coords[0], dtype=np.int32)
    cj = np.ascontiguousarray(coords[1], dtype=np.int32)
    v = np.ascontiguousarray(val, dtype=np.float64)
    Bc = np.ascontiguousarray(B, dtype=np.float64)
    out = np.empty((dims[0], Bc.shape[1]), dtype=np.float64)
    rc = _lib.timed_spmm(C.c_int64(dims[0]), C.c_int64(len(v)), ci.ctypes.data_as(C.c_void_p), cj.ctypes.data_as(C.c_void_p),
                         v.ctypes.data_as(C.c_void_p), Bc.ctypes.data_as(C.c_void_p), C.c_int64(Bc.shape[1]),
                         out.ctypes.data_as(C.c_void_p), C.c_int(threads))
    if rc != 0:
        raise RuntimeError("timed_spmm could not start its threads")
    return out
