"""Seeded synthetic inputs for BPDQ linear layers (logical tensors only).

This module draws the *inputs* of the quantized linear map: bit-planes B_i in {0,1},
fp16 group coefficients C_0..C_K and fp16 activations x.  It contains none of the
method's arithmetic (no decode, no dot product, no packing) so that both the CUDA
library's tests and the independent CPU checker can be fed the same numbers.

Everything comes from one counter-based generator: a value depends only on
(seed, tensor id, element counter), never on generation order.  That makes any
subset of rows reproducible on its own, and lets a device-side filler reproduce the
same tensors bit for bit.  The mixer is the published splitmix64 output function.

Value distributions (the paper's checkpoints are not available, only its layer
shapes are used):
  * plane bits   : iid Bernoulli(0.5); one 64-bit draw gives one 32-column word
                   (its high half), bit t of the word is column 32*w + t;
  * c0           : approximately N(0, 0.02): twelve 16-bit uniforms are summed in
                   integer arithmetic, centred, and scaled by one fp32 multiply;
  * c1, c2       : U(0.005, 0.05);  c3 and above: U(0.002, 0.02);  24-bit uniforms,
                   one fp32 multiply and one fp32 add, each rounded to nearest even;
  * x            : approximately N(0, 1), same twelve-uniform construction;
  all rounded once more to IEEE binary16 (round to nearest even).

No transcendental function is used, so a second implementation in another language
can agree exactly.
"""
from __future__ import annotations

import numpy as np

TENSOR_PLANES = 1
TENSOR_COEF = 2
TENSOR_X = 3

_GOLDEN = np.uint64(0x9E3779B97F4A7C15)
_M1 = np.uint64(0xBF58476D1CE4E5B9)
_M2 = np.uint64(0x94D049BB133111EB)

# fp32 constants, written as exact hex floats so that every implementation uses the same bits.
C0_SCALE = np.float32(float.fromhex("0x1.47ae14p-6")) * np.float32(2.0 ** -16)   # fl32(0.02) / 65536
X_SCALE = np.float32(2.0 ** -16)                                                  # 1 / 65536
U_LO_12 = np.float32(float.fromhex("0x1.47ae14p-8"))                              # fl32(0.005)
U_RANGE_12 = np.float32(float.fromhex("0x1.70a3d8p-5")) * np.float32(2.0 ** -24)  # (fl32(0.05)-fl32(0.005)) / 2^24
U_LO_3 = np.float32(float.fromhex("0x1.0624dep-9"))                               # fl32(0.002)
U_RANGE_3 = np.float32(float.fromhex("0x1.26e978p-6")) * np.float32(2.0 ** -24)   # (fl32(0.02)-fl32(0.002)) / 2^24
IH_CENTRE = 6 * 65535                                                             # mean of twelve 16-bit uniforms


def mix64(z: np.ndarray) -> np.ndarray:
    """splitmix64 output function on an array of uint64 (wrap-around arithmetic)."""
    z = np.asarray(z, dtype=np.uint64)
    with np.errstate(over="ignore"):
        z = (z ^ (z >> np.uint64(30))) * _M1
        z = (z ^ (z >> np.uint64(27))) * _M2
        z = z ^ (z >> np.uint64(31))
    return z


def stream_key(seed: int, tensor_id: int) -> np.uint64:
    """Key of one tensor's stream: mix64(seed XOR tensor_id * golden)."""
    with np.errstate(over="ignore"):
        k = np.array([np.uint64(seed & 0xFFFFFFFFFFFFFFFF)], dtype=np.uint64) ^ (
            np.array([tensor_id], dtype=np.uint64) * _GOLDEN)
    return mix64(k)[0]


def draw64(seed: int, tensor_id: int, counter: np.ndarray) -> np.ndarray:
    """64 random bits per counter: mix64(key + counter * golden)."""
    key = stream_key(seed, tensor_id)
    with np.errstate(over="ignore"):
        return mix64(key + np.asarray(counter, dtype=np.uint64) * _GOLDEN)


def _rows(out: int, rows) -> np.ndarray:
    if rows is None:
        return np.arange(out, dtype=np.uint64)
    rows = np.asarray(rows, dtype=np.int64)
    if rows.size and (rows.min() < 0 or rows.max() >= out):
        raise ValueError("row index out of range")
    return rows.astype(np.uint64)


def _irwin_hall_int(seed: int, tensor_id: int, elem: np.ndarray) -> np.ndarray:
    """Sum of twelve 16-bit uniforms minus its mean, as int64, from counters 4*elem + {0,1,2}."""
    elem = np.asarray(elem, dtype=np.uint64)
    total = np.zeros(elem.shape, dtype=np.int64)
    for part in range(3):
        w = draw64(seed, tensor_id, elem * np.uint64(4) + np.uint64(part))
        for q in range(4):
            total += ((w >> np.uint64(16 * q)) & np.uint64(0xFFFF)).astype(np.int64)
    return total - IH_CENTRE


def plane_words(seed: int, out: int, in_: int, K: int, rows=None) -> np.ndarray:
    """Logical plane words, uint32 [K][len(rows)][in/32]; bit t of word w is column 32*w+t."""
    if in_ % 32:
        raise ValueError("in must be a multiple of 32")
    r = _rows(out, rows)
    nw = in_ // 32
    i = np.arange(K, dtype=np.uint64)[:, None, None]
    q = (i * np.uint64(out) + r[None, :, None]) * np.uint64(nw) + np.arange(nw, dtype=np.uint64)[None, None, :]
    return (draw64(seed, TENSOR_PLANES, q) >> np.uint64(32)).astype(np.uint32)


def plane_bits(seed: int, out: int, in_: int, K: int, rows=None) -> np.ndarray:
    """Logical bit-planes, uint8 [K][len(rows)][in] with values 0/1 (plane i+1 of the paper at index i)."""
    w = plane_words(seed, out, in_, K, rows)
    t = np.arange(32, dtype=np.uint32)
    bits = ((w[..., None] >> t) & np.uint32(1)).astype(np.uint8)
    return bits.reshape(w.shape[0], w.shape[1], in_)


def coefficients(seed: int, out: int, in_: int, K: int, group: int, rows=None) -> np.ndarray:
    """fp16 bit patterns, uint16 [K+1][len(rows)][ceil(in/group)]; index 0 is the offset c0 (a last group may be short)."""
    r = _rows(out, rows)
    ng = -(-in_ // group)
    res = np.empty((K + 1, r.size, ng), dtype=np.uint16)
    g = np.arange(ng, dtype=np.uint64)[None, :]
    for i in range(K + 1):
        e = (np.uint64(i) * np.uint64(out) + r[:, None]) * np.uint64(ng) + g
        if i == 0:
            v = _irwin_hall_int(seed, TENSOR_COEF, e).astype(np.float32) * C0_SCALE
        else:
            u24 = (draw64(seed, TENSOR_COEF, e * np.uint64(4)) >> np.uint64(40)).astype(np.float32)
            lo, rng = (U_LO_12, U_RANGE_12) if i <= 2 else (U_LO_3, U_RANGE_3)
            v = (u24 * rng).astype(np.float32) + lo
        res[i] = v.astype(np.float32).astype(np.float16).view(np.uint16)
    return res


def activations(seed: int, M: int, in_: int, tokens=None) -> np.ndarray:
    """fp16 bit patterns of x, uint16 [M][in]; with `tokens` only those token rows, uint16 [len(tokens)][in]."""
    t = _rows(M, tokens)
    e = t[:, None] * np.uint64(in_) + np.arange(in_, dtype=np.uint64)[None, :]
    v = _irwin_hall_int(seed, TENSOR_X, e).astype(np.float32) * X_SCALE
    return v.astype(np.float16).view(np.uint16)


# ---------------------------------------------------------------------------------------------
# Workload shapes (out, in) of the paper's Qwen2.5 models; only the shapes are used.
# ---------------------------------------------------------------------------------------------
QWEN25_7B_LAYER = (("q", 3584, 3584), ("k", 512, 3584), ("v", 512, 3584), ("o", 3584, 3584),
                   ("gate", 18944, 3584), ("up", 18944, 3584), ("down", 3584, 18944))
QWEN25_72B_LAYER = (("q", 8192, 8192), ("k", 1024, 8192), ("v", 1024, 8192), ("o", 8192, 8192),
                    ("gate", 29568, 8192), ("up", 29568, 8192), ("down", 8192, 29568))


def linear_seed(base_seed: int, layer: int, linear_index: int, K: int) -> int:
    """Seed of one linear inside a multi-layer workload (plain integer packing, no hashing)."""
    return (base_seed << 32) ^ (layer << 16) ^ (linear_index << 8) ^ K
