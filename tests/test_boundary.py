"""The C-ABI library: it loads without a GPU, exports what the header declares, and rejects bad
arguments on the host (no compute call is made here)."""
import ctypes
import os
import re

import pytest

from paper_2510_08318_b200 import build as lib_build
from paper_2510_08318_b200 import linattn

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    lib_build.build()
    return linattn.load_library()


def declared_functions():
    text = open(os.path.join(ROOT, "include", "linattn.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(linattn_[a-z_]+)\s*\(", text)))


def test_header_and_binding_name_the_same_entry_points(lib):
    names = declared_functions()
    assert "linattn_create" in names and "linattn_forward" in names and "linattn_destroy" in names
    assert sorted(linattn.SIGNATURES) == names


def test_every_declared_symbol_is_exported(lib):
    raw = ctypes.CDLL(linattn.LIB_PATH)
    for name in declared_functions():
        assert hasattr(raw, name), f"{name} is declared in include/linattn.h but not exported"


def test_status_strings(lib):
    seen = {linattn.status_string(s) for s in range(7)}
    assert len(seen) == 7 and "ok" in seen
    assert linattn.status_string(99) == "unknown status"


def test_create_rejects_bad_arguments_before_touching_the_device(lib):
    h = ctypes.c_void_p()
    assert lib.linattn_create(None, 0, 12, 128, 1, 1024) == linattn.ERR_INVALID_ARG
    assert lib.linattn_create(ctypes.byref(h), 0, 0, 128, 1, 1024) == linattn.ERR_INVALID_ARG
    assert lib.linattn_create(ctypes.byref(h), 0, 12, 128, 0, 1024) == linattn.ERR_INVALID_ARG
    assert lib.linattn_create(ctypes.byref(h), 0, 12, 128, 1, 0) == linattn.ERR_INVALID_ARG
    assert lib.linattn_create(ctypes.byref(h), -1, 12, 128, 1, 1024) == linattn.ERR_INVALID_ARG
    assert lib.linattn_create(ctypes.byref(h), 0, 12, 96, 1, 1024) == linattn.ERR_UNSUPPORTED
    assert lib.linattn_create(ctypes.byref(h), 0, 12, 256, 1, 1024) == linattn.ERR_UNSUPPORTED
    assert not h.value


def test_null_context_is_rejected_everywhere(lib):
    assert lib.linattn_forward(None, 16, 16, 16, 16, 1, 1, 1, 64, linattn.BF16, None) == linattn.ERR_INVALID_ARG
    assert lib.linattn_forward_host(None, 16, 16, 16, 16, 1, 1, 1, 64, linattn.BF16, None) == linattn.ERR_INVALID_ARG
    assert lib.linattn_set_feature_map(None, 16, 16, 1, linattn.BF16, None) == linattn.ERR_INVALID_ARG
    assert lib.linattn_set_option(None, 0, 0) == linattn.ERR_INVALID_ARG
    assert lib.linattn_check(None, None) == linattn.ERR_INVALID_ARG
    assert lib.linattn_read_state(None, None, None, 1, None) == linattn.ERR_INVALID_ARG
    assert lib.linattn_destroy(None) == linattn.OK
    assert lib.linattn_last_launch_count(None) == 0
    assert lib.linattn_last_error(None) == b""


def test_missing_library_fails_loudly(monkeypatch, tmp_path):
    monkeypatch.setattr(linattn, "_lib", None)
    monkeypatch.setattr(linattn, "LIB_PATH", str(tmp_path / "nope.so"))
    with pytest.raises(ImportError):
        linattn.load_library()
