"""Pins of the reference checker's decode (variable grid, Eq. 1 / Eq. 7) against what the paper
and IEEE arithmetic fix.  CPU only."""
import itertools

import numpy as np
import pytest

import oracle
from paper_2602_04163_b200 import synth


def h(v) -> int:
    """fp16 bit pattern of a Python number, via numpy (an implementation independent of the checker)."""
    return int(np.array([v], dtype=np.float16).view(np.uint16)[0])


def f16(bits) -> np.ndarray:
    return np.asarray(bits, dtype=np.uint16).view(np.float16)


# ------------------------------------------------------------------ binary16 conversions
def test_half_to_float_exhaustive():
    allh = np.arange(65536, dtype=np.uint16)
    want = allh.view(np.float16).astype(np.float32)
    got = np.array([oracle.half_to_float(int(v)) for v in allh], dtype=np.float32)
    nan = np.isnan(want)
    assert np.array_equal(np.isnan(got), nan)
    assert np.array_equal(got[~nan].view(np.uint32), want[~nan].view(np.uint32))  # includes -0.0


def test_float_to_half_against_numpy():
    rng = np.random.default_rng(7)
    pats = [rng.integers(0, 2 ** 32, 200000, dtype=np.uint64).astype(np.uint32)]
    # every half value, its binary32 neighbours and the exact midpoints between adjacent halves
    allh = np.arange(0x7C00, dtype=np.uint16).view(np.float16).astype(np.float32)
    mid = ((allh[:-1].astype(np.float64) + allh[1:].astype(np.float64)) / 2).astype(np.float32)
    for base in (allh, mid, np.array([65504, 65519.99, 65520, 65536, 1e30, 2.0 ** -25, 2.0 ** -24,
                                      3 * 2.0 ** -26, 2.0 ** -26, 1e-40], dtype=np.float32)):
        u = base.view(np.uint32)
        pats += [u, u + np.uint32(1), u - np.uint32(1), u | np.uint32(0x80000000)]
    u = np.concatenate(pats)
    f = u.view(np.float32)
    with np.errstate(over="ignore"):
        want = f.astype(np.float16).view(np.uint16)
    got = np.array([oracle.float_to_half(float(v)) for v in f], dtype=np.uint16)
    nan = np.isnan(f)
    assert np.array_equal(got[~nan], want[~nan])
    assert np.all((got[nan] & 0x7C00) == 0x7C00) and np.all((got[nan] & 0x03FF) != 0)


# ------------------------------------------------------------------ hand-worked groups
def _golden_groups(golden_dir):
    rows = []
    with open(f"{golden_dir}/grid_handworked.txt") as fh:
        for line in fh:
            line = line.split("#")[0].strip()
            if not line:
                continue
            k, c, v = [p.split() for p in line.split("|")]
            rows.append((int(k[0]), [float(t) for t in c], [float(t) for t in v]))
    return rows


def test_handworked_groups(golden_dir):
    rows = _golden_groups(golden_dir)
    assert len(rows) >= 8
    for K, c, values in rows:
        assert len(c) == K + 1 and len(values) == 2 ** K
        g = 2 ** K  # one column per code
        bits = np.zeros((K, 1, g), dtype=np.uint8)
        for code in range(g):
            for i in range(K):
                bits[i, 0, code] = (code >> i) & 1
        coef = np.array([[[h(ci)]] for ci in c], dtype=np.uint16)
        w = oracle.dequant(bits, coef, g)
        assert np.array_equal(w[0], np.array([h(v) for v in values], dtype=np.uint16)), (K, c)


def test_group_index_and_plane_index():
    """REP repeats a coefficient over its g columns (G = floor(j/g)); plane i uses coefficient i."""
    K, out, in_, g = 3, 2, 12, 4
    coef = np.zeros((K + 1, out, in_ // g), dtype=np.uint16)
    vals = {}
    for i in range(K + 1):
        for r in range(out):
            for G in range(in_ // g):
                v = (1 + i) * 2.0 ** -3 + r * 4.0 + G * 16.0     # distinct, exactly summable
                coef[i, r, G] = h(v)
                vals[i, r, G] = v
    for i in range(K):
        bits = np.zeros((K, out, in_), dtype=np.uint8)
        bits[i] = 1
        w = f16(oracle.dequant(bits, coef, g)).astype(np.float64)
        for r in range(out):
            for j in range(in_):
                assert w[r, j] == vals[0, r, j // g] + vals[i + 1, r, j // g]


def test_cardinality_at_most_2_pow_K():
    for K, g in ((2, 128), (3, 128), (2, 64), (4, 32)):
        out, in_ = 24, 4 * g
        bits = synth.plane_bits(11, out, in_, K)
        coef = synth.coefficients(11, out, in_, K, g)
        w = oracle.dequant(bits, coef, g)
        for r in range(out):
            for G in range(in_ // g):
                assert len(set(w[r, G * g:(G + 1) * g].tolist())) <= 2 ** K
        # random bits over 128 columns hit every code, so the bound is attained
        if g >= 64:
            assert max(len(set(w[r, :g].tolist())) for r in range(out)) == 2 ** K


# ------------------------------------------------------------------ Proposition 1: uniform grid
@pytest.mark.parametrize("K", [2, 3, 4])
def test_uniform_grid_special_case(K):
    """c0 = -z*s, ci = s*2^(i-1) reproduces s*(q - z), q = sum bi 2^(i-1): plain integer dequant."""
    rng = np.random.default_rng(K)
    out, in_, g = 5, 96, 32
    q = rng.integers(0, 2 ** K, size=(out, in_))
    bits = np.stack([((q >> i) & 1).astype(np.uint8) for i in range(K)])
    e = rng.integers(1, 9, size=(out, in_ // g))
    z = rng.integers(0, 2 ** K, size=(out, in_ // g))
    s = 2.0 ** -e
    coef = np.empty((K + 1, out, in_ // g), dtype=np.uint16)
    coef[0] = (-(z * s)).astype(np.float16).view(np.uint16)
    for i in range(1, K + 1):
        coef[i] = (s * 2 ** (i - 1)).astype(np.float16).view(np.uint16)
    w = f16(oracle.dequant(bits, coef, g)).astype(np.float64)
    want = np.repeat(s, g, axis=1) * (q - np.repeat(z, g, axis=1))
    assert np.array_equal(w, want)

    # y through an all-integer route: every fp16 is an integer multiple of 2^-24.
    M = 3
    x = synth.activations(5, M, in_)
    xi = np.round(f16(x).astype(np.float64) * 2.0 ** 24).astype(np.int64)
    assert np.array_equal(xi.astype(np.float64) * 2.0 ** -24, f16(x).astype(np.float64))
    wi = (np.repeat(2 ** (8 - e), g, axis=1) * (q - np.repeat(z, g, axis=1))).astype(np.int64)  # w * 2^8
    y, a = oracle.linear(bits, coef, x, g)
    for m in range(M):
        for r in range(out):
            acc = sum(int(xi[m, j]) * int(wi[r, j]) for j in range(in_))
            assert y[m, r] == acc * 2.0 ** -32
            assert a[m, r] == sum(abs(int(xi[m, j]) * int(wi[r, j])) for j in range(in_)) * 2.0 ** -32


# ------------------------------------------------------------------ closed forms
@pytest.mark.parametrize("K", [1, 2, 3])
def test_all_zero_and_all_one_planes(K):
    out, in_, g = 16, 256, 128
    coef = synth.coefficients(3, out, in_, K, g)
    x = synth.activations(3, 2, in_)
    zero = np.zeros((K, out, in_), dtype=np.uint8)
    w0 = oracle.dequant(zero, coef, g)
    assert np.array_equal(w0, np.repeat(coef[0], g, axis=1))          # W^ = REP(C0), bit for bit
    y0, _ = oracle.linear(zero, coef, x, g)
    xs = f16(x).astype(np.float64).reshape(2, in_ // g, g).sum(axis=2)          # X_G per token
    want = xs @ f16(coef[0]).astype(np.float64).T
    assert np.allclose(y0, want, rtol=0, atol=1e-12)

    one = np.ones((K, out, in_), dtype=np.uint8)
    acc = f16(coef[0]).astype(np.float32)
    for i in range(1, K + 1):
        acc = (acc + f16(coef[i]).astype(np.float32)).astype(np.float32)       # ((c0+c1)+c2)+c3 in binary32
    assert np.array_equal(oracle.dequant(one, coef, g), np.repeat(acc.astype(np.float16).view(np.uint16), g, axis=1))


def test_negative_zero_offset_is_kept():
    """A clear bit adds nothing: c0 = -0.0 with all bits clear stays -0.0 (a '+0.0' would give +0.0)."""
    coef = np.array([[[0x8000]], [[h(0.5)]], [[h(0.25)]]], dtype=np.uint16)
    bits = np.zeros((2, 1, 4), dtype=np.uint8)
    bits[0, 0, 1] = 1
    bits[1, 0, 2] = 1
    bits[:, 0, 3] = 1
    assert oracle.dequant(bits, coef, 4)[0].tolist() == [0x8000, h(0.5), h(0.25), h(0.75)]


def test_rounding_ties_overflow_and_order():
    # binary16 spacing at 2048 is 2: 2049 is a tie and goes to the even neighbour 2048; 2051 -> 2052.
    def one(c, code):
        K = len(c) - 1
        bits = np.array([[[(code >> i) & 1]] for i in range(K)], dtype=np.uint8)
        coef = np.array([[[h(v)]] for v in c], dtype=np.uint16)
        return int(oracle.dequant(bits, coef, 1)[0, 0])

    assert one([2048, 1, 2], 0b01) == h(2048)
    assert one([2048, 1, 2], 0b11) == h(2052)
    assert one([2048, 1, 2], 0b10) == h(2050)
    # overflow: 65504 is the largest half; sums >= 65520 round to infinity, below it to 65504
    assert one([65504, 8, 16], 0b01) == h(65504)
    assert one([65504, 8, 16], 0b10) == 0x7C00
    assert one([-65504, -16, 8], 0b01) == 0xFC00
    # subnormal result kept: 2^-24 + 2^-24 = 2^-23
    assert one([2.0 ** -24, 2.0 ** -24, 0], 0b01) == 0x0002
    # order of the binary32 additions: ((2048 + 1) + 2^-13) + 2^-13 stays 2049 (two ties to even),
    # then the binary16 tie goes to 2048.  Any other order, or a wider accumulator, gives
    # 2049 + 2^-12 and rounds to 2050.
    assert one([2048, 1, 2.0 ** -13, 2.0 ** -13], 0b111) == h(2048)
    # cancellation is not reordered: (1024 + -1024) + 2^-20 = 2^-20 exactly
    assert one([1024, -1024, 2.0 ** -20], 0b11) == h(2.0 ** -20)
    # single rounding at the end: 1 + 2^-11 (a binary16 tie) + 2^-22 must round up, a decode that
    # rounded to binary16 after each plane would lose the first addend and stay at 1.0
    assert one([1, 2.0 ** -11, 2.0 ** -22], 0b11) == h(1 + 2.0 ** -10)


# ------------------------------------------------------------------ brute force on tiny shapes
def _table_decode(coef_f32, K):
    """Differently structured decode: build the 2^K values of a group first, then index."""
    table = []
    for code in range(2 ** K):
        acc = np.float32(coef_f32[0])
        for i in range(K):
            if (code >> i) & 1:
                acc = np.float32(acc + np.float32(coef_f32[i + 1]))
        table.append(np.array([acc], dtype=np.float32).astype(np.float16).view(np.uint16)[0])
    return table


@pytest.mark.parametrize("K,g", [(1, 32), (2, 16), (3, 8), (2, 32), (4, 16)])
def test_brute_force_tiny(K, g):
    rng = np.random.default_rng(100 + K)
    out, in_ = 3, 32
    # adversarial coefficients: mixed magnitudes and signs, some subnormal, drawn as raw fp16 patterns
    coef = rng.integers(0, 0x7C00, size=(K + 1, out, in_ // g)).astype(np.uint16)
    coef ^= (rng.integers(0, 2, size=coef.shape).astype(np.uint16) << 15)
    patterns = [np.zeros((K, out, in_), np.uint8), np.ones((K, out, in_), np.uint8)]
    for code in range(2 ** K):          # every code at every column
        b = np.empty((K, out, in_), np.uint8)
        for i in range(K):
            b[i] = (code >> i) & 1
        patterns.append(b)
    for j in range(in_):                # one-hot and its complement per plane
        for i in range(K):
            b = np.zeros((K, out, in_), np.uint8)
            b[i, :, j] = 1
            patterns += [b, 1 - b]
    patterns += [rng.integers(0, 2, size=(K, out, in_)).astype(np.uint8) for _ in range(40)]
    cf = f16(coef).astype(np.float32)
    tables = {(r, G): _table_decode(cf[:, r, G], K) for r in range(out) for G in range(in_ // g)}
    for b in patterns:
        w = oracle.dequant(b, coef, g)
        for r, j in itertools.product(range(out), range(in_)):
            code = sum(int(b[i, r, j]) << i for i in range(K))
            assert w[r, j] == tables[r, j // g][code]
