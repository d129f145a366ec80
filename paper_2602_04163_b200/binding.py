"""ctypes binding of libbpdq.so: argument marshalling only, same names as include/bpdq.h.

Every step of the hot path runs inside the library's CUDA kernels.  There is no CPU fallback:
if the library has not been built, importing a function from here raises.
PyTorch (or anything else) is only the owner of device buffers; this module takes raw
addresses (``tensor.data_ptr()``) and stream handles (``torch.cuda.current_stream().cuda_stream``).
"""
from __future__ import annotations

import ctypes
import os

import numpy as np

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG, "libbpdq.so")

OK, ERR_INVALID, ERR_UNSUPPORTED, ERR_ALLOC, ERR_CUDA, ERR_TIMEOUT = range(6)
KERNEL_AUTO, KERNEL_GEMV, KERNEL_GEMM, KERNEL_GEMV_SIMPLE, KERNEL_FEW = range(5)
GEMV_MAX_M = 16
FEW_MAX_M = 32
NOALLOC_MAX_OUT = 65536

EXPORTS = ("bpdq_packed_bytes", "bpdq_pack", "bpdq_unpack", "bpdq_create", "bpdq_dequant", "bpdq_linear",
           "bpdq_linear_ex", "bpdq_linear_host", "bpdq_set_gemv_max_m", "bpdq_set_few_max_m", "bpdq_read_blob", "bpdq_get_status",
           "bpdq_launch_count", "bpdq_destroy", "bpdq_quantize_datafree", "bpdq_truncate_planes", "bpdq_set_input_permutation", "bpdq_set_bias", "bpdq_gate_up_swiglu", "bpdq_probe_wait_limit", "bpdq_last_error", "bpdq_linear_noalloc", "bpdq_linear_batch", "bpdq_linear_batch_host")

_lib = None


class BpdqError(RuntimeError):
    def __init__(self, code: int, text: str):
        super().__init__(f"bpdq status {code}: {text}")
        self.code = code


def lib() -> ctypes.CDLL:
    """Loads libbpdq.so; raises if it is missing (build it with `python -m paper_2602_04163_b200.build`)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise ImportError(f"{LIB_PATH} is missing: the CUDA library has not been built "
                              "(python -m paper_2602_04163_b200.build); there is no fallback path")
        L = ctypes.CDLL(LIB_PATH)
        vp, i, u64 = ctypes.c_void_p, ctypes.c_int, ctypes.c_uint64
        L.bpdq_packed_bytes.argtypes = [i, i, i, i]
        L.bpdq_packed_bytes.restype = ctypes.c_size_t
        L.bpdq_pack.argtypes = [vp, vp, i, i, i, i, vp]
        L.bpdq_unpack.argtypes = [vp, i, i, i, i, vp, vp]
        L.bpdq_quantize_datafree.argtypes = [vp, i, i, i, i, ctypes.c_double, vp, vp]
        L.bpdq_truncate_planes.argtypes = [vp, vp, i, i, i, i, i, vp, vp]
        L.bpdq_create.argtypes = [ctypes.POINTER(vp), i, i, i, i, vp, u64, i]
        L.bpdq_dequant.argtypes = [vp, vp, vp]
        L.bpdq_linear.argtypes = [vp, vp, vp, i, vp]
        L.bpdq_linear_ex.argtypes = [vp, vp, vp, i, i, vp]
        L.bpdq_linear_host.argtypes = [vp, vp, vp, i, vp]
        L.bpdq_linear_batch.argtypes = [ctypes.POINTER(vp), ctypes.POINTER(vp), ctypes.POINTER(vp), i, i, vp]
        L.bpdq_linear_batch_host.argtypes = [ctypes.POINTER(vp), ctypes.POINTER(vp), ctypes.POINTER(vp), i, i, vp]
        L.bpdq_linear_noalloc.argtypes = [vp, i, i, i, i, vp, vp, i, vp]
        L.bpdq_set_gemv_max_m.argtypes = [vp, i]
        L.bpdq_set_few_max_m.argtypes = [vp, i]
        L.bpdq_set_input_permutation.argtypes = [vp, vp]
        L.bpdq_set_bias.argtypes = [vp, vp]
        L.bpdq_gate_up_swiglu.argtypes = [vp, vp, vp, vp, i, vp]
        L.bpdq_read_blob.argtypes = [vp, vp]
        L.bpdq_get_status.argtypes = [vp, vp]
        L.bpdq_probe_wait_limit.argtypes = [vp, vp]
        L.bpdq_launch_count.argtypes = [vp, ctypes.POINTER(u64)]
        L.bpdq_destroy.argtypes = [vp]
        L.bpdq_last_error.argtypes = []
        L.bpdq_last_error.restype = ctypes.c_char_p
        for name in EXPORTS:
            if name not in ("bpdq_packed_bytes", "bpdq_last_error"):
                getattr(L, name).restype = i
        _lib = L
    return _lib


def bpdq_last_error() -> str:
    return lib().bpdq_last_error().decode()


def _check(rc: int) -> None:
    if rc != OK:
        raise BpdqError(rc, bpdq_last_error())


def _np_ptr(a: np.ndarray) -> ctypes.c_void_p:
    return ctypes.c_void_p(a.ctypes.data)


def bpdq_packed_bytes(out: int, in_: int, K: int, group: int) -> int:
    return int(lib().bpdq_packed_bytes(out, in_, K, group))


def bpdq_pack(bits: np.ndarray, coef: np.ndarray, group: int) -> np.ndarray:
    """bits uint8 [K][out][in], coef uint16 [K+1][out][ceil(in/group)] -> blob (uint8 array)."""
    bits = np.ascontiguousarray(bits, dtype=np.uint8)
    coef = np.ascontiguousarray(coef, dtype=np.uint16)
    K, out, in_ = bits.shape
    if coef.shape != (K + 1, out, -(-in_ // group)):
        raise ValueError(f"coef shape {coef.shape} does not match bits {bits.shape} with group {group}")
    n = bpdq_packed_bytes(out, in_, K, group)
    if n == 0:
        raise BpdqError(ERR_UNSUPPORTED, f"unsupported shape out={out} in={in_} K={K} g={group}")
    blob = np.empty(n, dtype=np.uint8)
    _check(lib().bpdq_pack(_np_ptr(bits), _np_ptr(coef), out, in_, K, group, _np_ptr(blob)))
    return blob


def bpdq_unpack(blob: np.ndarray, out: int, in_: int, K: int, group: int):
    blob = np.ascontiguousarray(blob, dtype=np.uint8)
    if blob.size != bpdq_packed_bytes(out, in_, K, group) or blob.size == 0:
        raise BpdqError(ERR_INVALID, "blob size does not match the shape")
    bits = np.empty((K, out, in_), dtype=np.uint8)
    coef = np.empty((K + 1, out, -(-in_ // group)), dtype=np.uint16)
    _check(lib().bpdq_unpack(_np_ptr(blob), out, in_, K, group, _np_ptr(bits), _np_ptr(coef)))
    return bits, coef


def bpdq_quantize_datafree(w: np.ndarray, K: int, group: int, alpha: float = 1e-4):
    """w float32 [out][in] -> (bits uint8 [K][out][in], coef uint16 [K+1][out][ceil(in/group)])."""
    w = np.ascontiguousarray(w, dtype=np.float32)
    out, in_ = w.shape
    bits = np.empty((K, out, in_), dtype=np.uint8)
    coef = np.empty((K + 1, out, -(-in_ // group)), dtype=np.uint16)
    _check(lib().bpdq_quantize_datafree(_np_ptr(w), out, in_, K, group, alpha, _np_ptr(bits), _np_ptr(coef)))
    return bits, coef


def bpdq_truncate_planes(bits: np.ndarray, coef: np.ndarray, group: int, K2: int):
    """The view with the K2 most significant planes of (bits, coef)."""
    bits = np.ascontiguousarray(bits, dtype=np.uint8)
    coef = np.ascontiguousarray(coef, dtype=np.uint16)
    K, out, in_ = bits.shape
    bits2 = np.empty((K2, out, in_), dtype=np.uint8)
    coef2 = np.empty((K2 + 1, out, -(-in_ // group)), dtype=np.uint16)
    _check(lib().bpdq_truncate_planes(_np_ptr(bits), _np_ptr(coef), out, in_, K, group, K2, _np_ptr(bits2), _np_ptr(coef2)))
    return bits2, coef2


def bpdq_gate_up_swiglu(gate, up, x_ptr: int, h_ptr: int, M: int, stream: int = 0) -> None:
    """h = silu(x Wgate^T) * (x Wup^T) for two handles that share their input."""
    _check(lib().bpdq_gate_up_swiglu(gate._h, up._h, x_ptr, h_ptr, M, stream))


def bpdq_linear_noalloc(blob_ptr: int, out: int, in_: int, K: int, group: int, x_ptr: int, y_ptr: int, M: int,
                        stream: int = 0) -> None:
    """Look-up-table kernel on a caller-owned device blob; uses the library's static scratch, allocates nothing."""
    _check(lib().bpdq_linear_noalloc(blob_ptr, out, in_, K, group, x_ptr, y_ptr, M, stream))


def bpdq_linear_batch(handles, x_ptrs, y_ptrs, M: int, stream: int = 0) -> None:
    """Several independent linears (same K) in one launch of the look-up-table kernel."""
    n = len(handles)
    if not (n == len(x_ptrs) == len(y_ptrs)):
        raise ValueError("handles, x_ptrs and y_ptrs must have the same length")
    arr = ctypes.c_void_p * n
    _check(lib().bpdq_linear_batch(arr(*[h._h for h in handles]), arr(*x_ptrs), arr(*y_ptrs), n, M, stream))


def bpdq_linear_batch_host(handles, x_host_ptrs, y_host_ptrs, M: int, stream: int = 0) -> None:
    """bpdq_linear_batch with host buffers: copies in, one launch, copies out, one wait."""
    n = len(handles)
    if not (n == len(x_host_ptrs) == len(y_host_ptrs)):
        raise ValueError("handles, x_host_ptrs and y_host_ptrs must have the same length")
    arr = ctypes.c_void_p * n
    _check(lib().bpdq_linear_batch_host(arr(*[h._h for h in handles]), arr(*x_host_ptrs), arr(*y_host_ptrs), n, M, stream))


class Handle:
    """Owner of one bpdq_handle_t; the methods mirror the C entry points one to one."""

    def __init__(self, out: int, in_: int, K: int, group: int, host_blob: np.ndarray | None = None,
                 seed: int = 0, max_M: int = 1):
        self.out, self.in_, self.K, self.group, self.max_M = out, in_, K, group, max_M
        self._h = ctypes.c_void_p()
        ptr = None
        if host_blob is not None:
            host_blob = np.ascontiguousarray(host_blob, dtype=np.uint8)
            if host_blob.size != bpdq_packed_bytes(out, in_, K, group):
                raise BpdqError(ERR_INVALID, "blob size does not match the shape")
            ptr = _np_ptr(host_blob)
        _check(lib().bpdq_create(ctypes.byref(self._h), out, in_, K, group, ptr, seed & (2 ** 64 - 1), max_M))

    @property
    def packed_bytes(self) -> int:
        return bpdq_packed_bytes(self.out, self.in_, self.K, self.group)

    def bpdq_dequant(self, w_ptr: int, stream: int = 0) -> None:
        _check(lib().bpdq_dequant(self._h, w_ptr, stream))

    def bpdq_linear(self, x_ptr: int, y_ptr: int, M: int, stream: int = 0) -> None:
        _check(lib().bpdq_linear(self._h, x_ptr, y_ptr, M, stream))

    def bpdq_linear_ex(self, x_ptr: int, y_ptr: int, M: int, kernel: int, stream: int = 0) -> None:
        _check(lib().bpdq_linear_ex(self._h, x_ptr, y_ptr, M, kernel, stream))

    def bpdq_linear_host(self, x_host_ptr: int, y_host_ptr: int, M: int, stream: int = 0) -> None:
        _check(lib().bpdq_linear_host(self._h, x_host_ptr, y_host_ptr, M, stream))

    def bpdq_set_gemv_max_m(self, m: int) -> None:
        _check(lib().bpdq_set_gemv_max_m(self._h, m))

    def bpdq_set_few_max_m(self, m: int) -> None:
        _check(lib().bpdq_set_few_max_m(self._h, m))

    def bpdq_set_input_permutation(self, perm) -> None:
        if perm is None:
            _check(lib().bpdq_set_input_permutation(self._h, None))
        else:
            perm = np.ascontiguousarray(perm, dtype=np.int32)
            if perm.shape != (self.in_,):
                raise ValueError("perm must have one entry per input channel")
            _check(lib().bpdq_set_input_permutation(self._h, _np_ptr(perm)))

    def bpdq_set_bias(self, bias_bits) -> None:
        if bias_bits is None:
            _check(lib().bpdq_set_bias(self._h, None))
        else:
            bias_bits = np.ascontiguousarray(bias_bits, dtype=np.uint16)
            if bias_bits.shape != (self.out,):
                raise ValueError("bias must have one entry per output row")
            _check(lib().bpdq_set_bias(self._h, _np_ptr(bias_bits)))

    def bpdq_read_blob(self) -> np.ndarray:
        blob = np.empty(self.packed_bytes, dtype=np.uint8)
        _check(lib().bpdq_read_blob(self._h, _np_ptr(blob)))
        return blob

    def bpdq_get_status(self, stream: int = 0) -> None:
        _check(lib().bpdq_get_status(self._h, stream))

    def bpdq_probe_wait_limit(self, stream: int = 0) -> None:
        _check(lib().bpdq_probe_wait_limit(self._h, stream))

    def bpdq_launch_count(self) -> int:
        c = ctypes.c_uint64()
        _check(lib().bpdq_launch_count(self._h, ctypes.byref(c)))
        return int(c.value)

    def bpdq_destroy(self) -> None:
        if self._h:
            h, self._h = self._h, ctypes.c_void_p()
            _check(lib().bpdq_destroy(h))

    def __del__(self):
        try:
            self.bpdq_destroy()
        except Exception:
            pass
