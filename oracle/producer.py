"""Data-free BPDQ producer -- TEST INFRASTRUCTURE ONLY (part of the reference checker).

The initialisation of the paper's quantizer, restated without calibration data, in plain numpy binary64:

  * Bit-plane selection (Section 3.2 "Variable Grid Initialization", Eq. 5): every (row, group of g columns) of W goes
    through an asymmetric round-to-nearest quantizer to an unsigned 8-bit code Z; Z = sum_i 2^i P_i; the planes kept
    are the K most significant ones, B_i = P_{7-K+i} for i = 1..K (B_K is the most significant).
  * Scalar coefficient fitting (Eq. 6) with U_loc = I (no calibration data, hence no Hessian): per row and group the
    (K+1)-vector c minimising || [1, b_1, .., b_K] c - w ||_2, from the normal equations.

Readings where the paper is silent: the affine quantizer takes minimum and maximum per (row, group), scale =
(max - min) / 255, code = rint((w - min) / scale) (ties to even), a constant group gets code 0 and scale 1; the damping
factor alpha = 1e-4, which the paper applies "to the diagonal", is added to the diagonal of the normal matrix as
alpha * trace / (K + 1), so that a plane that is constant within a group leaves the system solvable; coefficients are
rounded once to binary16 for storage.

`truncate_planes` is the multi-precision view the paper's closing section points to (serving several precisions from
one stored model) under this reading: the K' most significant planes are kept with their coefficients, and every
dropped plane contributes half its coefficient to the offset (its expected value when set and clear are equally
likely); sums in binary32 in plane order, one rounding to binary16.
"""
from __future__ import annotations

import numpy as np


def rtn_uint8(w: np.ndarray, group: int):
    """Per (row, group) asymmetric round-to-nearest to codes 0..255.  Returns (Z uint8 [out][in], lo, scale [out][in/g])."""
    w = np.asarray(w, dtype=np.float64)
    out, in_ = w.shape
    assert in_ % group == 0
    wg = w.reshape(out, in_ // group, group)
    lo = wg.min(axis=2)
    hi = wg.max(axis=2)
    scale = (hi - lo) / 255.0
    scale = np.where(scale > 0, scale, 1.0)
    z = np.rint((wg - lo[:, :, None]) / scale[:, :, None])
    z = np.clip(z, 0, 255).astype(np.uint8)
    return z.reshape(out, in_), lo, scale


def msb_planes(z: np.ndarray, K: int) -> np.ndarray:
    """bits[i-1] = B_i = P_{7-K+i} of Z, i = 1..K (Eq. 5 and the selection rule below it)."""
    z = np.asarray(z, dtype=np.uint8)
    return np.stack([(z >> (7 - K + i)) & 1 for i in range(1, K + 1)]).astype(np.uint8)


def fit_coefficients(w: np.ndarray, bits: np.ndarray, group: int, alpha: float = 1e-4) -> np.ndarray:
    """Eq. 6 with U_loc = I, per (row, group): returns binary64 [K+1][out][in/g] (index 0 is the offset)."""
    w = np.asarray(w, dtype=np.float64)
    K, out, in_ = bits.shape
    ng = in_ // group
    c = np.zeros((K + 1, out, ng))
    for r in range(out):
        for G in range(ng):
            cols = slice(G * group, (G + 1) * group)
            B = np.concatenate([np.ones((group, 1)), bits[:, r, cols].T.astype(np.float64)], axis=1)   # g x (K+1)
            N = B.T @ B
            N = N + alpha * (np.trace(N) / (K + 1)) * np.eye(K + 1)
            c[:, r, G] = np.linalg.solve(N, B.T @ w[r, cols])
    return c


def produce(w: np.ndarray, K: int, group: int, alpha: float = 1e-4):
    """W -> (bits uint8 [K][out][in], coef uint16 [K+1][out][in/g] binary16 bit patterns)."""
    z, _, _ = rtn_uint8(w, group)
    bits = msb_planes(z, K)
    c = fit_coefficients(w, bits, group, alpha)
    return bits, c.astype(np.float32).astype(np.float16).view(np.uint16)


def truncate_planes(bits: np.ndarray, coef: np.ndarray, K2: int):
    """(bits, coef) with K planes -> the view with the K2 most significant planes (see the module text)."""
    K = bits.shape[0]
    assert 1 <= K2 <= K and coef.shape[0] == K + 1
    drop = K - K2
    cf = coef.view(np.float16).astype(np.float32)
    c0 = cf[0].copy()
    for i in range(1, drop + 1):                      # plane order, binary32, each step rounded
        c0 = (c0 + np.float32(0.5) * cf[i]).astype(np.float32)
    new = np.concatenate([c0[None].astype(np.float16).view(np.uint16), coef[drop + 1:]], axis=0)
    return np.ascontiguousarray(bits[drop:]), np.ascontiguousarray(new)
