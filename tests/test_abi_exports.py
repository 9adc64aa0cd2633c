"""The shared library loads and exports every symbol include/slonn.h declares.
No compute call is made, so this runs without a GPU."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "slonn.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(slonn_[a-z_0-9]+)\s*\(", text)))


def test_header_declares_the_boundary_calls():
    names = declared_symbols()
    for must in ("slonn_build", "slonn_run", "slonn_run_host", "slonn_free", "slonn_workspace_bytes"):
        assert must in names


def test_library_exports_every_declared_symbol():
    from paper_2204_08400_b200 import build_ext, binding
    path = build_ext.build()
    lib = ctypes.CDLL(path)
    for name in declared_symbols():
        assert hasattr(lib, name), name
    assert sorted(binding.EXPORTS) == declared_symbols()
    assert binding.version() == 1
    assert binding.strerror(-5) == "budget out of range"


def test_binding_fails_loudly_without_the_library(monkeypatch, tmp_path):
    from paper_2204_08400_b200 import binding
    monkeypatch.setattr(binding, "_lib", None)
    monkeypatch.setattr(binding, "LIB_PATH", str(tmp_path / "missing.so"))
    with pytest.raises(RuntimeError):
        binding.version()
