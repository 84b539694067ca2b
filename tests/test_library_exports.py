"""The C-ABI shared library builds for sm_100a, loads, and exports every symbol the header declares."""
import ctypes
import os
import re
import shutil

import pytest

from paper_2503_23186_b200 import binding, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared_symbols():
    text = open(os.path.join(ROOT, "include", "b2c.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(b2c_[a-z0-9_]+)\s*\(", text)))


@pytest.fixture(scope="module")
def so_path():
    if not os.path.exists(build.SO) or build.needs_build():
        if shutil.which("nvcc") is None and not os.path.exists("/usr/local/cuda/bin/nvcc"):
            pytest.skip("nvcc not available and library not built")
        build.build()
    return build.SO


def test_header_symbols_are_exported(so_path):
    lib = ctypes.CDLL(so_path)
    declared = _declared_symbols()
    assert len(declared) >= 25
    missing = [s for s in declared if not hasattr(lib, s)]
    assert not missing, missing
    assert sorted(binding.EXPORTS) == declared


def test_status_strings_and_create_without_device(so_path):
    lib = binding.lib()
    for code in range(9):
        assert lib.b2c_status_string(code)
    assert lib.b2c_status_string(0) == b"ok"
    import torch
    if not torch.cuda.is_available():
        handle = ctypes.c_void_p()
        assert lib.b2c_create(ctypes.byref(handle), 0) != 0   # no device: an error status, not a crash
        assert not handle
    assert lib.b2c_bn_relu_bwd_workspace_bytes(64) == 2 * 64 * 8
    assert lib.b2c_create(None, 0) == 1
