"""Pins of the reference checker's linear map y = x * W^T and of its blob reader.  CPU only."""
import numpy as np
import pytest

import oracle
from paper_2602_04163_b200 import synth


def f16(bits):
    return np.asarray(bits, dtype=np.uint16).view(np.float16)


@pytest.mark.parametrize("K,g,out,in_,M", [(2, 128, 48, 384, 1), (3, 128, 40, 256, 3), (2, 64, 24, 192, 2),
                                            (4, 256, 8, 512, 1)])
def test_linear_matches_float64_matmul(K, g, out, in_, M):
    """Special case that reduces to a library routine: dequantize, then a float64 matrix product.
    Non-square shapes with M != out catch a transposed operand or a swapped output index."""
    bits = synth.plane_bits(21, out, in_, K)
    coef = synth.coefficients(21, out, in_, K, g)
    x = synth.activations(22, M, in_)
    w = f16(oracle.dequant(bits, coef, g)).astype(np.float64)
    xf = f16(x).astype(np.float64)
    y, a = oracle.linear(bits, coef, x, g)
    assert y.shape == (M, out)
    assert np.allclose(y, xf @ w.T, rtol=1e-12, atol=1e-12)
    assert np.allclose(a, np.abs(xf) @ np.abs(w).T, rtol=1e-12, atol=1e-12)
    assert np.all(a >= np.abs(y) - 1e-12)


def test_linear_one_hot_activation_reads_one_column():
    """x = e_j picks column j of W^: y[0, r] = W^[r, j] exactly."""
    K, g, out, in_ = 2, 128, 16, 256
    bits = synth.plane_bits(1, out, in_, K)
    coef = synth.coefficients(1, out, in_, K, g)
    w = f16(oracle.dequant(bits, coef, g)).astype(np.float64)
    for j in (0, 1, 127, 128, 255):
        x = np.zeros((1, in_), dtype=np.float16)
        x[0, j] = 1.0
        y, a = oracle.linear(bits, coef, x.view(np.uint16), g)
        assert np.array_equal(y[0], w[:, j])
        assert np.array_equal(a[0], np.abs(w[:, j]))


def test_linear_add_only_identity():
    """y_r = sum_G [ c0*X_G + sum_i ci * S_i ],  S_i = sum of x over the set bits of plane i
    (the add-only form the paper names for custom hardware) agrees with the definition up to the
    one binary16 rounding of each weight."""
    K, g, out, in_ = 3, 128, 32, 512
    bits = synth.plane_bits(9, out, in_, K)
    coef = synth.coefficients(9, out, in_, K, g)
    x = synth.activations(9, 1, in_)
    y, a = oracle.linear(bits, coef, x, g)
    xf = f16(x).astype(np.float64)[0]
    cf = f16(coef).astype(np.float64)
    alt = np.zeros(out)
    for G in range(in_ // g):
        xs = xf[G * g:(G + 1) * g]
        alt += cf[0, :, G] * xs.sum()
        for i in range(K):
            alt += cf[i + 1, :, G] * (bits[i, :, G * g:(G + 1) * g] * xs).sum(axis=1)
    assert np.all(np.abs(alt - y[0]) <= 2.0 ** -11 * a[0] + 1e-12)


def test_unpack_reads_documented_layout():
    """Build a blob by hand from the layout description and read it back."""
    K, g, out, in_ = 2, 128, 32, 256
    bits = synth.plane_bits(4, out, in_, K)
    coef = synth.coefficients(4, out, in_, K, g)
    nblk = in_ // 128
    planes = np.zeros((nblk, K, out, 16), dtype=np.uint8)
    for b in range(nblk):
        for i in range(K):
            for r in range(out):
                for p in range(16):
                    L = (p + r) % 16
                    k, q = divmod(L, 4)
                    planes[b, i, r, p] = sum(int(bits[i, r, 128 * b + 32 * k + 8 * (t % 4) + 2 * q + t // 4]) << t
                                             for t in range(8))
    cblob = np.transpose(coef, (2, 0, 1)).copy()          # [G][i][r]
    blob = np.concatenate([planes.reshape(-1), cblob.reshape(-1).view(np.uint8)])
    b2, c2 = oracle.unpack(blob, out, in_, K, g)
    assert np.array_equal(b2, bits) and np.array_equal(c2, coef)


def test_short_last_group():
    """in not a multiple of g: G = floor(j / g) still names every column's group, and the last group is the short one
    (the paper's W2-G256 setting meets a 29568-channel input, 115.5 groups).  Hand-made dyadic coefficients: every
    candidate value is exact, and the columns either side of the last group boundary must use different ones."""
    K, g, out, in_ = 2, 256, 2, 384                       # one whole group and one of 128 columns
    ng = 2
    c = np.array([[0.5, 0.25, 0.125], [-1.0, 2.0, 4.0]])   # [group][c0, c1, c2]
    coef = np.zeros((K + 1, out, ng), dtype=np.uint16)
    for G in range(ng):
        for i in range(K + 1):
            coef[i, :, G] = np.float16(c[G, i] * np.array([1.0, -2.0])).view(np.uint16)   # row 1: the same times -2
    bits = np.zeros((K, out, in_), dtype=np.uint8)
    bits[0, :, 1::2] = 1                                   # plane 1 on odd columns
    bits[1, :, 2::4] = 1                                   # plane 2 on columns 2, 3 mod 4
    bits[1, :, 3::4] = 1
    w = oracle.dequant(bits, coef, g).view(np.float16).astype(np.float64)
    for j in (0, 1, 2, 3, 254, 255, 256, 257, 258, 259, 382, 383):
        G = j // g
        want = c[G, 0] + c[G, 1] * bits[0, 0, j] + c[G, 2] * bits[1, 0, j]
        assert w[0, j] == want and w[1, j] == -2.0 * want, j
    assert w[0, 255] == 0.875 and w[0, 256] == -1.0 and w[0, 383] == 5.0     # ... worked out by hand
    # the linear map through the same tensors equals a binary64 product with the decoded weights
    x = synth.activations(5, 3, in_)
    y, a = oracle.linear(bits, coef, x, g)
    xf = x.view(np.float16).astype(np.float64)
    assert np.allclose(y, xf @ w.T, rtol=1e-13, atol=1e-13) and np.allclose(a, np.abs(xf) @ np.abs(w).T, rtol=1e-13, atol=1e-13)
    # and the blob reader finds ceil(in / g) coefficient groups behind the planes
    planes = np.zeros((in_ // 128, K, out, 16), dtype=np.uint8)
    for b in range(in_ // 128):
        for i in range(K):
            for r in range(out):
                for p in range(16):
                    k, q = divmod((p + r) % 16, 4)
                    planes[b, i, r, p] = sum(int(bits[i, r, 128 * b + 32 * k + 8 * (t % 4) + 2 * q + t // 4]) << t for t in range(8))
    blob = np.concatenate([planes.reshape(-1), np.transpose(coef, (2, 0, 1)).copy().reshape(-1).view(np.uint8)])
    b2, c2 = oracle.unpack(blob, out, in_, K, g)
    assert np.array_equal(b2, bits) and np.array_equal(c2, coef)
