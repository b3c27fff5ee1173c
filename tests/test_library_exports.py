"""The C-ABI library builds for sm_100a, loads without a GPU, and exports every symbol the header
declares (no compute call is made here)."""

import ctypes
import os
import re

from paper_2503_14649_b200 import binding, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    text = open(os.path.join(ROOT, "include", "rago.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(rago_[a-z0-9_]+)\s*\(", text)))


def test_header_symbols_are_exported():
    path = build.build()
    lib = ctypes.CDLL(path)
    names = _declared()
    assert len(names) >= 12
    for n in names:
        assert hasattr(lib, n), n
    assert set(names) == set(binding.EXPORTS)


def test_host_only_calls_work_without_a_device():
    lib = binding.lib()
    assert binding.rago_kernel_launches() >= 0
    assert lib.rago_last_error() is not None
    # argument errors are detected on the host
    out = ctypes.c_size_t()
    assert lib.rago_flat_workspace_bytes(10, 64, 2, 0, ctypes.byref(out)) == 1
    assert b"sizes" in lib.rago_last_error()
    assert lib.rago_flat_workspace_bytes(10_000_000, 1024, 256, 100, ctypes.byref(out)) == 0
    assert out.value >= 256 * 148 * 256 * 8  # 256 queries x 148 database ranges x 256 keys
    assert lib.rago_search_workspace_bytes(None, 1, 1, 1, ctypes.byref(out)) == 1
    assert lib.rago_index_free(None) == 0


def test_binding_refuses_to_run_without_the_library(monkeypatch, tmp_path):
    monkeypatch.setattr(binding, "_lib", None)
    monkeypatch.setattr(binding, "LIB_PATH", str(tmp_path / "missing.so"))
    try:
        binding.lib()
    except RuntimeError as e:
        assert "no CPU fallback" in str(e)
    else:
        raise AssertionError("a missing library must be an error")
