"""The C ABI library loads without a GPU and exports every symbol the public header declares."""
import os
import re

from paper_2609_22098_b200 import binding, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "treespark.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(ts_[a-z_]+)\s*\(", text)))


def test_library_builds_loads_and_exports_the_header():
    build.build()
    lib = binding.load_library()
    names = declared_symbols()
    assert set(names) == set(binding.EXPORTS), names
    for n in names:
        assert getattr(lib, n) is not None


def test_missing_library_is_an_error_not_a_fallback(monkeypatch):
    monkeypatch.setattr(binding, "_lib", None)
    monkeypatch.setattr(binding, "LIB_PATH", os.path.join(ROOT, "no_such_library.so"))
    import pytest
    with pytest.raises(RuntimeError):
        binding.load_library()


def test_host_side_argument_checks_need_no_device():
    lib = binding.load_library()
    import ctypes as C
    out = C.c_void_p()
    assert lib.ts_create(None, C.byref(out)) == -1
    assert b"null" in lib.ts_last_error_string()
    cfg = binding.TsConfig(100, 4, 8, 32, 16, 1, 0, 0, 0, 0, 0, 0.67, -0.46, -10, 10, None)
    assert lib.ts_create(C.byref(cfg), C.byref(out)) == -2          # K > 16 is unsupported
    cfg = binding.TsConfig(100, 4, 8, 4, 16, 1, 0, 1, 0, 0, 0, 0.67, -0.46, -10, 10, None)
    assert lib.ts_create(C.byref(cfg), C.byref(out)) == -2          # mixed dtypes
    assert lib.ts_workspace_bytes(None, 1) == 0
