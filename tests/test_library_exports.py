"""The C boundary without a GPU: the library builds for sm_100a, loads, and exports every
function that include/qsparse.h declares; argument checks that need no device work."""
import ctypes as C
import os
import re

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_functions():
    text = open(os.path.join(ROOT, "include", "qsparse.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(qs_[a-z_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported():
    from paper_1906_02367_b200 import binding as B
    L = B.lib()
    names = declared_functions()
    assert len(names) >= 15
    for n in names:
        assert hasattr(L, n), n
    assert sorted(B.EXPORTS) == names


def test_null_and_bad_arguments_are_rejected_on_the_host():
    from paper_1906_02367_b200 import binding as B
    L = B.lib()
    assert L.qs_init(None, 1, 10, 1, 4, 0, 0, None) == B.QS_INVALID_ARG
    h = C.c_void_p()
    for args in [(0, 10, 1, 4, 0), (33, 10, 1, 4, 0), (2, 0, 1, 4, 0), (2, 10, 11, 4, 0), (2, 10, 0, 4, 0),
                 (2, 10, 1, 0, 0), (2, 10, 1, 70000, 0), (2, 10, 1, 4, 7), (2, 2**32, 1, 4, 0),
                 (2, 2**32 - 4095, 1, 4, 0)]:          # d beyond what the 32-bit tile arithmetic of the kernels covers
        R, d, k, s, op = args
        assert L.qs_init(C.byref(h), R, d, k, s, op, 0, None) == B.QS_INVALID_ARG and not h.value
    assert L.qs_wire_words(None) < 0 and L.qs_total_k(None) < 0
    assert L.qs_sync_status(None) == B.QS_INVALID_ARG
    assert L.qs_last_error(None) == b"null context"
    L.qs_destroy(None)


def test_build_flags_target_blackwell_without_fma():
    from paper_1906_02367_b200 import build
    flags = " ".join(build.NVCC_FLAGS)
    assert "arch=compute_100a,code=sm_100a" in flags and "-fmad=false" in flags
