"""The C-ABI library loads without a GPU and exports every symbol include/algproj.h declares."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    text = open(os.path.join(ROOT, "include", "algproj.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(alg_[a-z0-9_]+)\s*\(", text)))


def test_header_symbols_are_exported():
    from paper_2609_32814_b200 import binding, build
    build.build()
    lib = ctypes.CDLL(binding.LIB_PATH)
    names = _declared()
    assert len(names) >= 18
    for n in names:
        assert hasattr(lib, n), f"{n} declared in algproj.h but not exported"
    assert sorted(binding.EXPORTS) == names


def test_status_strings_and_argument_errors_need_no_gpu():
    from paper_2609_32814_b200 import binding
    L = binding.lib()
    assert L.alg_status_string(0) == b"ok"
    assert L.alg_status_string(5) == b"row type outside [0, q)"
    h = ctypes.c_void_p()
    w = (ctypes.c_int32 * 2)(128, 128)
    wp = ctypes.cast(w, ctypes.c_void_p)
    assert L.alg_proj_create(ctypes.byref(h), 0, wp, wp, 1, 0, None, 0) == 1      # q < 1
    assert L.alg_proj_create(ctypes.byref(h), 257, wp, wp, 1, 0, None, 0) == 1    # q > ALG_MAX_Q_LARGE
    w33 = ctypes.cast((ctypes.c_int32 * 33)(*([128] * 33)), ctypes.c_void_p)
    assert L.alg_proj_create(ctypes.byref(h), 33, w33, w33, 0, 0, None, 0) == 2   # q > ALG_MAX_Q: bf16 operands only
    assert L.alg_proj_create(ctypes.byref(h), 2, None, wp, 1, 0, None, 0) == 1    # NULL widths
    assert L.alg_proj_create(ctypes.byref(h), 2, wp, wp, 7, 0, None, 0) == 1      # bad dtype
    assert L.alg_proj_create(ctypes.byref(h), 2, wp, wp, 1, 2, None, 0) == 1      # custom table without keep
    w3 = (ctypes.c_int32 * 3)(128, 128, 128)
    w3p = ctypes.cast(w3, ctypes.c_void_p)
    assert L.alg_proj_create(ctypes.byref(h), 3, w3p, w3p, 1, 3, None, 0) == 1    # tensor-power law needs q = 2^L
    bad = (ctypes.c_int32 * 2)(128, 0)
    assert L.alg_proj_create(ctypes.byref(h), 2, ctypes.cast(bad, ctypes.c_void_p), wp, 1, 0, None, 0) == 1
    assert L.alg_proj_destroy(None) == 1
    assert L.alg_launch_count() >= 0


def test_missing_library_is_loud(monkeypatch, tmp_path):
    from paper_2609_32814_b200 import binding
    monkeypatch.setattr(binding, "_lib", None)
    monkeypatch.setattr(binding, "LIB_PATH", str(tmp_path / "nope.so"))
    with pytest.raises(FileNotFoundError):
        binding.lib()
