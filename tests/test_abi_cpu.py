"""Host-side checks that need no GPU: the CUDA library builds for sm_100a, loads, and
exports every entry point the header declares; the binding mirrors the header."""
import ctypes
import os
import re

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    text = open(os.path.join(ROOT, "include", "dqrm.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(dqrm_[a-z0-9_]+)\s*\(", text)))


def test_library_builds_and_exports_every_declared_symbol():
    from paper_2410_20046_b200 import build, binding

    path = build.build()
    lib = ctypes.CDLL(path)
    names = _declared()
    assert len(names) >= 12
    for n in names:
        assert hasattr(lib, n), f"{n} declared in dqrm.h but not exported"
    assert sorted(binding.SIGNATURES) == names


def test_status_strings_and_argument_checks_without_a_device():
    from paper_2410_20046_b200 import binding

    lib = binding.load_library()
    assert lib.dqrm_status_string(0) == b"ok"
    for code in (-1, -2, -3, -4, -5):
        assert lib.dqrm_status_string(code) not in (b"ok", b"unknown status")
    assert lib.dqrm_status_string(-99) == b"unknown status"
    h = ctypes.c_void_p()
    off = (ctypes.c_int64 * 3)(0, 5, 5)           # not strictly increasing
    assert lib.dqrm_create(ctypes.byref(h), 2, 16, off) == binding.ERR_INVALID_ARG
    off = (ctypes.c_int64 * 3)(0, 5, 9)
    assert lib.dqrm_create(ctypes.byref(h), 2, 18, off) == binding.ERR_INVALID_ARG   # D % 4
    assert lib.dqrm_create(ctypes.byref(h), 0, 16, off) == binding.ERR_INVALID_ARG
    assert lib.dqrm_create(None, 2, 16, off) == binding.ERR_INVALID_ARG
    assert lib.dqrm_workspace_bytes(None, 10, 10) == 0
    assert lib.dqrm_destroy(None) == 0


def test_missing_library_raises_instead_of_falling_back(tmp_path):
    import pytest
    from paper_2410_20046_b200 import binding

    with pytest.raises(ImportError):
        binding.load_library(str(tmp_path / "nope.so"))
