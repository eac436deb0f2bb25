"""The C-ABI library loads without a GPU and exports every symbol include/rocs.h declares."""
import ctypes
import os
import re

import pytest

import __graft_entry__ as entry
from paper_2607_27744_b200 import binding

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    if not os.path.exists(binding.LIB_PATH):
        entry.build()
    return ctypes.CDLL(binding.LIB_PATH)


def _declared():
    text = open(os.path.join(ROOT, "include", "rocs.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(rocs_[a-z0-9_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(lib):
    names = _declared()
    assert {"rocs_ikbo_linear", "rocs_dca_attention", "rocs_glm_interaction", "rocs_plan_create"} <= set(names)
    for n in names:
        assert hasattr(lib, n), f"{n} declared in rocs.h but not exported"
    assert set(binding.EXPORTS) == set(names)


def test_host_only_helpers(lib):
    lib.rocs_status_string.restype = ctypes.c_char_p
    assert lib.rocs_status_string(0) == b"ok"
    assert b"align" in lib.rocs_status_string(-2)
    lib.rocs_padded_ld.restype = ctypes.c_int64
    lib.rocs_padded_ld.argtypes = [ctypes.c_int64, ctypes.c_int]
    assert lib.rocs_padded_ld(250, 0) == 256 and lib.rocs_padded_ld(256, 0) == 256
    assert lib.rocs_padded_ld(5, 1) == 8 and lib.rocs_padded_ld(0, 1) == 0


def test_null_arguments_are_rejected_before_any_cuda_call(lib):
    assert lib.rocs_plan_create(None, 1, 1, None, None, None) == -1
    assert lib.rocs_ikbo_linear(None, 0, 1, 1, 1, None, 0, None, 0, None, 0, None, 0, None, 0, None, 0, None, 0, None) == -1
    assert lib.rocs_set_path(7) == -1 and lib.rocs_set_path(0) == 0


def test_binding_fails_loudly_without_the_library(monkeypatch, tmp_path):
    monkeypatch.setattr(binding, "_lib", None)
    monkeypatch.setattr(binding, "LIB_PATH", str(tmp_path / "missing.so"))
    with pytest.raises(RuntimeError, match="no fallback"):
        binding.lib()
