"""B200-native sparse x dense tensor contractions driven by per-dimension storage attributes
(dense, compressed-unique, compressed-nonunique, singleton): COO -> CSR/DCSR/CSF packing, SpMV, SpMM,
TTV, TTM and MTTKRP as hand-written sm_100a CUDA kernels behind a C ABI (include/comet.h).

This package is the thin Python binding of that library; see `binding` for the calls.
"""
from .binding import (D, CU, CN, S, CometError, Handle, SpTensor, default_handle, load_library, pack, validate,  # noqa: F401
                      spmv, spmm, elementwise_mul, spmm_from_host, ttv_symbolic, ttv, ttm_symbolic, ttm, mttkrp, reorder,
                      EXPORTS, LIB_PATH)
