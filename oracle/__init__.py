"""ctypes front end of the BPDQ reference checker -- TEST INFRASTRUCTURE ONLY.

The checker itself is ``bpdq_oracle.cpp`` in this directory (single-threaded C++, no CUDA).
This file only compiles it with g++ on first use and marshals numpy arrays.  It must never
be imported by the product package; only tests, the smoke check and the benchmark's
CPU-baseline leg use it.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "bpdq_oracle.cpp")
_LIB = os.path.join(_HERE, "liboracle_bpdq.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the checker.  No fast-math, no FMA contraction: binary32 steps stay as written."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        cmd = ["g++", "-std=c++17", "-O2", "-fPIC", "-shared", "-ffp-contract=off", "-fno-fast-math",
               "-Wall", "-Wextra", "-o", _LIB + ".tmp", _SRC]
        subprocess.run(cmd, check=True)
        os.replace(_LIB + ".tmp", _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        i64, p = ctypes.c_int64, ctypes.c_void_p
        lib.oracle_half_to_float.argtypes = [ctypes.c_uint16]
        lib.oracle_half_to_float.restype = ctypes.c_float
        lib.oracle_float_to_half.argtypes = [ctypes.c_float]
        lib.oracle_float_to_half.restype = ctypes.c_uint16
        lib.oracle_dequant.argtypes = [p, p, i64, i64, ctypes.c_int, i64, p]
        lib.oracle_linear.argtypes = [p, p, p, i64, i64, ctypes.c_int, i64, i64, p, p]
        lib.oracle_unpack.argtypes = [p, i64, i64, ctypes.c_int, i64, p, p]
        lib.oracle_linear_perm.argtypes = [p, p, p, p, i64, i64, ctypes.c_int, i64, i64, p, p]
        lib.oracle_silu.argtypes = [ctypes.c_double]
        lib.oracle_silu.restype = ctypes.c_double
        lib.oracle_swiglu.argtypes = [p, p, i64, p]
        lib.oracle_add_bias.argtypes = [p, p, i64, i64]
        for f in (lib.oracle_dequant, lib.oracle_linear, lib.oracle_unpack, lib.oracle_linear_perm, lib.oracle_swiglu, lib.oracle_add_bias):
            f.restype = ctypes.c_int
        _lib = lib
    return _lib


def _c(a: np.ndarray, dtype) -> np.ndarray:
    a = np.ascontiguousarray(a, dtype=dtype)
    return a


def _ptr(a: np.ndarray):
    return ctypes.c_void_p(a.ctypes.data)


def half_to_float(h: int) -> float:
    return float(_load().oracle_half_to_float(int(h)))


def float_to_half(f: float) -> int:
    return int(_load().oracle_float_to_half(float(f)))


def dequant(bits: np.ndarray, coef: np.ndarray, group: int) -> np.ndarray:
    """bits uint8 [K][out][in], coef uint16 [K+1][out][ceil(in/group)] -> fp16 bit patterns uint16 [out][in]."""
    bits = _c(bits, np.uint8)
    coef = _c(coef, np.uint16)
    K, out, in_ = bits.shape
    assert coef.shape == (K + 1, out, -(-in_ // group)), (coef.shape, bits.shape, group)
    w = np.empty((out, in_), dtype=np.uint16)
    rc = _load().oracle_dequant(_ptr(bits), _ptr(coef), out, in_, K, group, _ptr(w))
    if rc:
        raise ValueError("oracle_dequant rejected its arguments")
    return w


def linear(bits: np.ndarray, coef: np.ndarray, x: np.ndarray, group: int):
    """Returns (y, a): float64 [M][out] each; a = sum_j |x_j * w_j| is the error scale."""
    bits = _c(bits, np.uint8)
    coef = _c(coef, np.uint16)
    x = _c(x, np.uint16)
    K, out, in_ = bits.shape
    M = x.shape[0]
    assert x.shape == (M, in_)
    assert coef.shape == (K + 1, out, -(-in_ // group))
    y = np.empty((M, out), dtype=np.float64)
    a = np.empty((M, out), dtype=np.float64)
    rc = _load().oracle_linear(_ptr(bits), _ptr(coef), _ptr(x), out, in_, K, group, M, _ptr(y), _ptr(a))
    if rc:
        raise ValueError("oracle_linear rejected its arguments")
    return y, a


def unpack(blob: np.ndarray, out: int, in_: int, K: int, group: int):
    """Device blob (uint8) -> (bits uint8 [K][out][in], coef uint16 [K+1][out][ceil(in/group)])."""
    blob = _c(blob, np.uint8)
    need = out * in_ * K // 8 + out * (-(-in_ // group)) * (K + 1) * 2
    assert blob.size == need, (blob.size, need)
    bits = np.empty((K, out, in_), dtype=np.uint8)
    coef = np.empty((K + 1, out, -(-in_ // group)), dtype=np.uint16)
    rc = _load().oracle_unpack(_ptr(blob), out, in_, K, group, _ptr(bits), _ptr(coef))
    if rc:
        raise ValueError("oracle_unpack rejected its arguments")
    return bits, coef


def linear_perm(bits: np.ndarray, coef: np.ndarray, x: np.ndarray, perm: np.ndarray, group: int):
    """y[m,r] = sum_j x[m, perm[j]] * w[r,j]: the stored columns are a reordering of the input channels.  Returns (y, a)."""
    bits = _c(bits, np.uint8)
    coef = _c(coef, np.uint16)
    x = _c(x, np.uint16)
    perm = _c(perm, np.int64)
    K, out, in_ = bits.shape
    M = x.shape[0]
    assert x.shape == (M, in_) and perm.shape == (in_,)
    y = np.empty((M, out), dtype=np.float64)
    a = np.empty((M, out), dtype=np.float64)
    rc = _load().oracle_linear_perm(_ptr(bits), _ptr(coef), _ptr(x), _ptr(perm), out, in_, K, group, M, _ptr(y), _ptr(a))
    if rc:
        raise ValueError("oracle_linear_perm rejected its arguments (perm must be a permutation)")
    return y, a


def silu(v: float) -> float:
    return float(_load().oracle_silu(float(v)))


def swiglu(gate: np.ndarray, up: np.ndarray) -> np.ndarray:
    """h = silu(gate) * up, elementwise in binary64."""
    gate = _c(gate, np.float64)
    up = _c(up, np.float64)
    assert gate.shape == up.shape
    h = np.empty(gate.shape, dtype=np.float64)
    if _load().oracle_swiglu(_ptr(gate), _ptr(up), gate.size, _ptr(h)):
        raise ValueError("oracle_swiglu rejected its arguments")
    return h


def add_bias(y: np.ndarray, bias: np.ndarray) -> np.ndarray:
    """y + float(bias) per output row, bias as binary16 bit patterns [out]."""
    y = np.array(y, dtype=np.float64, order="C")
    bias = _c(bias, np.uint16)
    assert y.ndim == 2 and bias.shape == (y.shape[1],)
    if _load().oracle_add_bias(_ptr(y), _ptr(bias), y.shape[0], y.shape[1]):
        raise ValueError("oracle_add_bias rejected its arguments")
    return y
