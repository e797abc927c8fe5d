"""The C-ABI library builds, loads and exports every entry point the header declares."""
import ctypes
import os
import re

import pytest

from paper_2505_13204_b200 import binding, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    text = open(os.path.join(ROOT, "include", "aasd.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(aasd_[a-z_]+)\s*\(", text)))


def test_header_declares_the_three_calls():
    names = _declared()
    for n in ("aasd_align_sample", "aasd_draft", "aasd_verify", "aasd_select", "aasd_append",
              "aasd_step"):
        assert n in names


def test_library_exports_every_declared_symbol():
    lib = ctypes.CDLL(build.build())
    for n in _declared():
        assert hasattr(lib, n), n
    assert sorted(binding.EXPORTS) == _declared()


def test_status_strings_and_workspace_size_without_gpu():
    lib = binding.load_library()
    assert lib.aasd_status_str(0) == b"ok"
    assert b"workspace" in lib.aasd_status_str(4)
    n = ctypes.c_size_t()
    assert lib.aasd_workspace_bytes(4096, 512, ctypes.byref(n)) == 0
    small = n.value
    assert lib.aasd_workspace_bytes(8192, 512, ctypes.byref(n)) == 0
    assert n.value > small > 0
    assert lib.aasd_workspace_bytes(-1, 0, ctypes.byref(n)) == 1


def test_struct_sizes_match_the_header_layout():
    # natural alignment of the C structs in include/aasd.h
    assert ctypes.sizeof(binding.AlignParams) == 48
    assert ctypes.sizeof(binding.VerifyParams) == 56
    assert ctypes.sizeof(binding.DraftParams) == 24
    assert ctypes.sizeof(binding.Counters) == 64


def test_no_cpu_fallback(monkeypatch):
    import torch
    if torch.cuda.is_available():
        pytest.skip("a GPU is present")
    with pytest.raises(RuntimeError):
        binding.Context()
