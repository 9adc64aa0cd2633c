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


def test_build_refuses_layer_inputs_too_wide_to_stage_before_touching_the_device():
    """A dense layer input wider than SLONN_MAX_INPUT_WIDTH (or one that leaves no room for an activator layer's
    node bitmap beside it) is refused with SLONN_ERR_DIM by the argument checks, which run before any device call,
    so this needs no GPU: the weight pointers are never followed."""
    from paper_2204_08400_b200 import binding as sl
    fake = 0x1000                                   # aligned, non-null, never dereferenced
    for dims, act in (([57604, 8], [0]), ([8, 57604, 8], [0, 0]), ([57000, 400000, 8], [1, 0])):
        with pytest.raises(sl.SlonnError) as e:
            sl.slonn_build(dims, act, sl.SLONN_F32, [fake] * (len(dims) - 1), [fake] * (len(dims) - 1),
                           calib_dense=None, K=2, L=1)
        assert e.value.code == sl.ERR["DIM"], dims
