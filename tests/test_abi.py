"""The C-ABI library loads without a GPU and exports every function include/comet.h declares; the
binding refuses to run without a CUDA device instead of falling back to anything."""
import ctypes
import os
import re

import pytest
import torch

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_functions():
    text = open(os.path.join(ROOT, "include", "comet.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(comet_[a-z0-9_]+)\s*\(", text)))


def test_header_declares_the_boundary():
    names = declared_functions()
    for must in ["comet_pack", "comet_spmv", "comet_spmm", "comet_ttv", "comet_ttm", "comet_mttkrp"]:
        assert must in names


def test_library_exports_every_declared_symbol():
    import paper_2102_05187_b200 as comet
    from paper_2102_05187_b200 import build
    build.build()
    lib = ctypes.CDLL(comet.LIB_PATH)
    for name in declared_functions():
        assert hasattr(lib, name), f"libcomet.so does not export {name}"
    assert sorted(comet.EXPORTS) == declared_functions()
    lib.comet_status_string.restype = ctypes.c_char_p
    assert lib.comet_status_string(0) == b"ok" and b"duplicate" in lib.comet_status_string(-4)


def test_struct_layout_matches_header():
    from paper_2102_05187_b200.binding import SpTensorStruct
    # int32 x2, int64 x4, int32 x4, int32 x4, ptr x4, int64 x4, ptr x4, int64 x4, ptr, int64, ptr
    assert ctypes.sizeof(SpTensorStruct) == 8 + 32 + 16 + 16 + 32 + 32 + 32 + 32 + 8 + 8 + 8


@pytest.mark.skipif(torch.cuda.is_available(), reason="checks the behaviour of a box without a GPU")
def test_no_cpu_fallback():
    import paper_2102_05187_b200 as comet
    with pytest.raises(RuntimeError):
        comet.Handle()
    with pytest.raises(ValueError):
        comet.pack([torch.zeros(1, dtype=torch.int32)] * 2, torch.zeros(1, dtype=torch.float64), (2, 2), (0, 1), (0, 1),
                   handle=object())
