"""The C-ABI library builds, loads, and exports every symbol include/clada.h declares (no GPU needed)."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    text = open(os.path.join(ROOT, "include", "clada.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(clada_[a-z_0-9]+)\s*\(", text)))


@pytest.fixture(scope="module")
def lib():
    from paper_2502_19078_b200 import build
    return ctypes.CDLL(build.build())


def test_header_declares_the_four_path_calls():
    names = _declared()
    for must in ("clada_prefix_select", "clada_cogload", "clada_adjust_threshold", "clada_sparse_ffn_decode"):
        assert must in names


def test_every_declared_symbol_is_exported(lib):
    for name in _declared():
        assert hasattr(lib, name), f"{name} declared in clada.h but not exported"


def test_host_only_calls(lib):
    assert lib.clada_version() >= 100
    lib.clada_status_string.restype = ctypes.c_char_p
    assert lib.clada_status_string(0) == b"ok"
    for code in range(-7, 0):
        assert lib.clada_status_string(code) not in (b"ok", b"unknown status")
    assert lib.clada_status_string(-99) == b"unknown status"


def test_host_validation_rejects_before_touching_the_device(lib):
    # NULL pointers and bad sizes are refused on the host: nothing is enqueued, no GPU is needed.
    assert lib.clada_cogload(None, 0, 1, 8, 8, None, None, None, None, None) == -1
    assert lib.clada_select(None, 1, 8, None, 1, None, None, None, None) == -1
    assert lib.clada_adjust_threshold(None, None, None, ctypes.c_float(0), ctypes.c_float(0), None, None, 1, 1,
                                      None, None) == -1
    assert lib.clada_sparse_ffn_decode(None, None, 1, None, None, 1, None, 0, None, None, None, None, 0, None,
                                       None) == -1
    assert lib.clada_workspace_init(None, 0, None) == -1


def test_binding_refuses_to_run_without_the_library(monkeypatch):
    from paper_2502_19078_b200 import binding
    monkeypatch.setattr(binding, "_lib", None)
    monkeypatch.setattr(binding, "LIB_PATH", os.path.join(ROOT, "no_such_dir", "libclada.so"))
    with pytest.raises(binding.CladaError):
        binding.load()


def test_binding_exposes_the_same_names():
    from paper_2502_19078_b200 import binding
    for name in _declared():
        if name in ("clada_status_string", "clada_last_cuda_error"):
            continue
        assert hasattr(binding, name), name
