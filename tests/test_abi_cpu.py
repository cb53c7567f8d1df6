"""The C-ABI library loads without a GPU and exports what the header declares."""
import ctypes
import os
import re

import pytest

from paper_2509_26538_b200 import binding, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    build.build_library()
    return binding.lib()


def _declared_functions():
    text = open(os.path.join(ROOT, "include", "hilberta.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(hilberta_[a-z_0-9]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(lib):
    names = _declared_functions()
    assert set(names) == set(binding.SYMBOLS)
    for n in names:
        assert hasattr(lib, n), n


def test_binding_constants_match_the_header():
    """Element types, error codes and export selectors are spelled twice (header, binding): same values."""
    text = open(os.path.join(ROOT, "include", "hilberta.h")).read()
    defs = {m.group(1): int(m.group(2).strip("()"), 0)
            for m in re.finditer(r"^#define\s+HILBERTA_([A-Z0-9_]+)\s+(\(?-?\d+\)?)\s", text, flags=re.M)}
    for name in ("BF16", "FP32", "FP8_E4M3", "ERR_INVALID", "ERR_UNSUPPORTED", "ERR_ARCH", "ERR_CUDA", "ERR_NOMEM",
                 "ERR_BUFFER", "ERR_UNBOUND", "ERR_TIMEOUT", "EXPORT_HIL_D2T", "EXPORT_HIL_T2D", "EXPORT_PHYS2ORIG",
                 "EXPORT_ORIG2PHYS", "EXPORT_SHARED_RUNS", "EXPORT_WINDOWS", "EXPORT_NNZ", "EXPORT_INFO", "EXPORT_LAUNCH_CLOCK"):
        assert name in defs, name
        assert getattr(binding, name) == defs[name], name
    assert len({defs["BF16"], defs["FP32"], defs["FP8_E4M3"]}) == 3


def test_version_and_status_strings(lib):
    assert lib.hilberta_version() == 100
    seen = set()
    for code in range(0, -9, -1):
        s = lib.hilberta_status_string(code).decode()
        assert s and s != "unknown status"
        seen.add(s)
    assert len(seen) == 9
    assert lib.hilberta_status_string(-99).decode() == "unknown status"


def test_argument_validation_needs_no_device(lib):
    h = ctypes.c_void_p()
    bad = [
        (0, 0, 4, 0, 0, 0), (8, 8, 0, 0, 0, 0), (8, 8, 16, 0, 0, -1), (8, 8, 16, 0, -2, 0),
    ]
    for args in bad:
        assert lib.hilberta_plan(*args, ctypes.byref(h)) == binding.ERR_INVALID
    assert lib.hilberta_plan(2048, 16, 16, 0, 0, 0, ctypes.byref(h)) == binding.ERR_UNSUPPORTED
    assert lib.hilberta_plan(12, 12, 48, 0, 0, 0, ctypes.byref(h)) == binding.ERR_INVALID  # 48 does not divide 16*16
    assert lib.hilberta_plan(8, 16, 16, 0, 10, 0, ctypes.byref(h)) == binding.ERR_INVALID  # shared side > H
    assert lib.hilberta_plan(8, 8, 5, 0, 0, 0, ctypes.byref(h)) == binding.ERR_INVALID
    assert lib.hilberta_plan(8, 8, 16, 0, 3, 0, ctypes.byref(h)) == binding.ERR_INVALID
    assert lib.hilberta_plan(8, 8, 16, 0, 10, 0, ctypes.byref(h)) == binding.ERR_INVALID
    assert lib.hilberta_plan(8, 8, 16, 0, 0, 0, None) == binding.ERR_INVALID
    assert lib.hilberta_plan_destroy(None) == 0
    assert lib.hilberta_forward(None, None, None, None, None, None) == binding.ERR_INVALID
    assert lib.hilberta_permute(None, None, None, 1, 8, 0, None) == binding.ERR_INVALID
    assert lib.hilberta_plan_export(None, 0, None, 0, None) == binding.ERR_INVALID


def test_missing_library_fails_loudly(monkeypatch):
    monkeypatch.setattr(binding, "_lib", None)
    monkeypatch.setattr(binding, "LIB_PATH", "/nonexistent/libhilberta.so")
    with pytest.raises(ImportError):
        binding.lib()
