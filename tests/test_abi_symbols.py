"""The C-ABI library loads without a GPU and exports every symbol include/llma.h declares."""
import ctypes
import os
import re

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_library_exports_header_symbols():
    import __graft_entry__ as G
    G.build()
    from paper_2304_04487_b200 import LIB_PATH, lib
    from paper_2304_04487_b200.binding import EXPORTS
    header = open(os.path.join(ROOT, "include", "llma.h")).read()
    declared = set(re.findall(r"\b(llma_[a-z0-9_]+)\s*\(", header))
    assert declared, "no declarations found"
    L = ctypes.CDLL(LIB_PATH)
    for name in declared:
        assert hasattr(L, name), f"{name} declared in llma.h but not exported"
    assert declared == set(EXPORTS)
    assert lib().llma_strerror(0) == b"ok"
    assert b"capacity" in lib().llma_strerror(-4)


def test_argument_errors_need_no_gpu():
    from paper_2304_04487_b200 import lib
    L = lib()
    assert L.llma_create(None, None, None, None) == -1
    assert L.llma_prefill(None, 0, None, 0) == -1
    assert L.llma_destroy(None) == 0
