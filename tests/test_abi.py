"""The C-ABI library loads without a GPU and exports every symbol that include/bpdq.h declares."""
import ctypes
import os
import re

import pytest

from paper_2602_04163_b200 import binding

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "bpdq.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"BPDQ_API[^;(]*?\b(bpdq_\w+)\s*\(", text)))


def test_header_declares_the_expected_entry_points():
    names = declared_symbols()
    for must in ("bpdq_create", "bpdq_dequant", "bpdq_linear", "bpdq_destroy", "bpdq_pack", "bpdq_unpack",
                 "bpdq_packed_bytes", "bpdq_last_error"):
        assert must in names
    assert set(names) == set(binding.EXPORTS)


def test_library_exports_every_declared_symbol():
    L = ctypes.CDLL(binding.LIB_PATH)
    for name in declared_symbols():
        assert hasattr(L, name), name


def test_host_side_argument_checks_need_no_gpu():
    L = binding.lib()
    assert L.bpdq_destroy(None) == binding.OK
    assert L.bpdq_dequant(None, None, None) == binding.ERR_INVALID
    assert L.bpdq_linear(None, None, None, 1, None) == binding.ERR_INVALID
    assert "null handle" in binding.bpdq_last_error()
    h = ctypes.c_void_p()
    assert L.bpdq_create(ctypes.byref(h), 100, 256, 2, 128, None, 0, 1) == binding.ERR_UNSUPPORTED
    assert not h.value
    assert L.bpdq_create(ctypes.byref(h), 128, 256, 2, 128, None, 0, 0) == binding.ERR_INVALID
    assert L.bpdq_create(None, 128, 256, 2, 128, None, 0, 1) == binding.ERR_INVALID
    assert L.bpdq_pack(None, None, 16, 128, 2, 128, None) == binding.ERR_INVALID


def test_create_without_device_fails_cleanly():
    import torch
    if torch.cuda.is_available():
        pytest.skip("a device is present")
    h = ctypes.c_void_p()
    rc = binding.lib().bpdq_create(ctypes.byref(h), 128, 256, 2, 128, None, 0, 1)
    assert rc in (binding.ERR_UNSUPPORTED, binding.ERR_CUDA) and not h.value
