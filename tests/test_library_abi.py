"""The C-ABI library builds for sm_100a, loads without a GPU and exports every symbol that
include/szo.h declares; host-side argument validation works without launching anything."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def libpath():
    from paper_2406_02913_b200 import build
    return build.build()


def _declared():
    text = open(os.path.join(ROOT, "include", "szo.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(szo_[a-z0-9_]+)\s*\(", text)))


def test_header_symbols_are_exported(libpath):
    lib = ctypes.CDLL(libpath)
    names = _declared()
    assert len(names) >= 20
    for n in names:
        assert hasattr(lib, n), f"{n} declared in szo.h but not exported"


def test_binding_signature_table_matches_header():
    from paper_2406_02913_b200 import binding
    assert binding.exported_symbols() == _declared()


def test_status_strings_and_host_validation(libpath):
    lib = ctypes.CDLL(libpath)
    lib.szo_status_string.restype = ctypes.c_char_p
    lib.szo_last_error.restype = ctypes.c_char_p
    assert lib.szo_status_string(0) == b"SZO_OK"
    assert lib.szo_status_string(-8) == b"SZO_ERR_TIMEOUT"
    assert lib.szo_version() >= 100
    # k < 0 is rejected before any CUDA call
    lib.szo_perturb.argtypes = [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int64,
                                ctypes.c_int64, ctypes.c_uint64, ctypes.c_uint64, ctypes.c_float,
                                ctypes.c_void_p]
    assert lib.szo_perturb(None, None, None, -1, 0, 0, 0, 1.0, None) == -1
    assert b"k < 0" in lib.szo_last_error()
    # misaligned pointers are rejected on the host
    assert lib.szo_perturb(4, 4, 4, 8, 0, 0, 0, 1.0, None) == -3
    # quantize: K not a multiple of G
    lib.szo_quantize.argtypes = [ctypes.c_void_p, ctypes.c_int, ctypes.c_int64, ctypes.c_int64,
                                 ctypes.c_int32, ctypes.c_int, ctypes.c_void_p, ctypes.c_void_p,
                                 ctypes.c_void_p, ctypes.c_void_p]
    assert lib.szo_quantize(16, 0, 4, 100, 64, 1, 16, 16, 16, None) == -2
    # select: k > n, and the workspace-size query needs no device
    lib.szo_select_mask.argtypes = [ctypes.c_void_p, ctypes.c_int64, ctypes.c_int64, ctypes.c_void_p,
                                    ctypes.c_void_p, ctypes.POINTER(ctypes.c_size_t), ctypes.c_void_p]
    nb = ctypes.c_size_t(0)
    assert lib.szo_select_mask(16, 10, 11, 16, None, ctypes.byref(nb), None) == -1
    assert lib.szo_select_mask(16, 1 << 20, 10, 16, None, ctypes.byref(nb), None) == 0 and nb.value > 0
