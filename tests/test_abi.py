"""The C-ABI library loads and exports every entry point that include/seer.h declares
(no compute calls are made here; runs without a GPU)."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    text = open(os.path.join(ROOT, "include", "seer.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(seer_[a-z_]+)\s*\(", text)))


def test_header_declares_the_four_operations():
    names = _declared()
    for n in ("seer_gate_select", "seer_sparse_decode", "seer_dense_decode", "seer_kcomp_append"):
        assert n in names


def test_library_exports_every_declared_symbol():
    from paper_2506_08889_b200 import binding, build
    build.build()
    L = ctypes.CDLL(binding.LIB_PATH)
    for name in _declared():
        assert hasattr(L, name), name
    assert sorted(binding.EXPORTS) == _declared()


def test_create_without_a_device_fails_cleanly():
    import torch
    if torch.cuda.is_available():
        pytest.skip("a GPU is present")
    from paper_2506_08889_b200 import binding
    with pytest.raises(binding.SeerError):
        binding.Context(0)
    assert binding.lib().seer_status_string(binding.SEER_ERR_BAD_INDEX).decode().startswith("block index")


def test_binding_refuses_to_run_without_the_library(monkeypatch):
    from paper_2506_08889_b200 import binding
    monkeypatch.setattr(binding, "_lib", None)
    monkeypatch.setattr(binding, "LIB_PATH", "/nonexistent/libseer.so")
    with pytest.raises(RuntimeError):
        binding.lib()


def test_product_package_never_touches_the_oracle():
    pkg = os.path.join(ROOT, "paper_2506_08889_b200")
    for dirpath, _, files in os.walk(pkg):
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".h")):
                src = open(os.path.join(dirpath, f)).read()
                assert "oracle" not in src.lower(), f
