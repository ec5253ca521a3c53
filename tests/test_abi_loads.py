"""The C-ABI library builds for sm_100a, loads without a GPU, and exports every entry point
that include/a2sgd.h declares (no compute call is made here)."""
import ctypes
import os
import re

import pytest

from paper_2006_07405_b200 import binding, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    text = open(os.path.join(ROOT, "include", "a2sgd.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(a2sgd_[a-z_0-9]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    path = build.build()
    lib = ctypes.CDLL(path)
    names = _declared()
    assert {"a2sgd_create", "a2sgd_encode", "a2sgd_global_average", "a2sgd_decode_update", "a2sgd_step"} <= set(names)
    for name in names:
        assert hasattr(lib, name), f"{name} declared in a2sgd.h but not exported"


def test_binding_names_match_the_header():
    for name in _declared():
        if name == "a2sgd_status_string":
            assert hasattr(binding, "status_string")
        else:
            assert hasattr(binding, name), f"binding lacks {name}"


def test_status_strings_and_host_side_argument_checks():
    lib = binding.lib()
    assert binding.status_string(0) == "ok"
    for code in range(-7, 0):
        assert binding.status_string(code) != "unknown status"
    assert binding.status_string(-99) == "unknown status"
    # NULL context / NULL out pointer are rejected before any CUDA call
    assert lib.a2sgd_create(None, 10, 1, 0, 0) == binding.ERR_ARG
    assert lib.a2sgd_step(None, None, 0, None, 0, None, 0, 0.1, None) == binding.ERR_ARG
    assert lib.a2sgd_destroy(None) == binding.OK


def test_missing_library_fails_loudly(monkeypatch):
    monkeypatch.setattr(binding, "_lib", None)
    monkeypatch.setattr(binding, "LIB_PATH", "/nonexistent/liba2sgd.so")
    with pytest.raises(RuntimeError, match="no CPU fallback"):
        binding.lib()
