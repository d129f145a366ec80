"""Pins of the checker's steps around the linear map: input-channel reordering, gated unit, bias, and the data-free
producer (bit-plane selection of Eq. 5, coefficient fit of Eq. 6 with U_loc = I).  CPU only."""
import numpy as np
import pytest

import oracle
from oracle import producer
from paper_2602_04163_b200 import synth


def f16(bits):
    return np.asarray(bits, dtype=np.uint16).view(np.float16)


# ---- reordering ---------------------------------------------------------------------------------------------------------
def _group_perm(in_, g, seed):
    """Groups moved as wholes (what Group-Aware Reordering does) and shuffled inside."""
    rng = np.random.default_rng(seed)
    order = rng.permutation(in_ // g)
    return np.concatenate([G * g + rng.permutation(g) for G in order]).astype(np.int64)


@pytest.mark.parametrize("K,g,out,in_,M", [(2, 128, 24, 384, 2), (3, 64, 16, 256, 1)])
def test_perm_equals_plain_map_on_gathered_activations(K, g, out, in_, M):
    bits, coef, x = synth.plane_bits(3, out, in_, K), synth.coefficients(3, out, in_, K, g), synth.activations(4, M, in_)
    perm = _group_perm(in_, g, 5)
    y, a = oracle.linear_perm(bits, coef, x, perm, g)
    y2, a2 = oracle.linear(bits, coef, x[:, perm], g)                     # the gather done outside, then the pinned plain map
    assert np.array_equal(y, y2) and np.array_equal(a, a2)
    yi, _ = oracle.linear_perm(bits, coef, x, np.arange(in_), g)          # identity: the plain map
    assert np.array_equal(yi, oracle.linear(bits, coef, x, g)[0])
    assert not np.array_equal(y, yi)


def test_perm_leaves_the_layer_function_unchanged():
    """Scattering the stored columns back to channel order gives a matrix whose plain product with x is y:
    W_orig[:, perm[j]] = W^[:, j]  =>  y = x W_orig^T (float64 matmul, a library routine)."""
    K, g, out, in_, M = 2, 128, 12, 256, 3
    bits, coef, x = synth.plane_bits(6, out, in_, K), synth.coefficients(6, out, in_, K, g), synth.activations(7, M, in_)
    perm = _group_perm(in_, g, 8)
    w = f16(oracle.dequant(bits, coef, g)).astype(np.float64)
    w_orig = np.empty_like(w)
    w_orig[:, perm] = w
    y, _ = oracle.linear_perm(bits, coef, x, perm, g)
    assert np.allclose(y, f16(x).astype(np.float64) @ w_orig.T, rtol=1e-12, atol=1e-12)


def test_perm_rejects_what_is_not_a_permutation():
    bits, coef, x = synth.plane_bits(1, 4, 128, 2), synth.coefficients(1, 4, 128, 2, 128), synth.activations(1, 1, 128)
    bad = np.arange(128)
    bad[5] = 6
    with pytest.raises(ValueError):
        oracle.linear_perm(bits, coef, x, bad, 128)


# ---- gated unit and bias ----------------------------------------------------------------------------------------------
def test_silu_closed_forms():
    assert oracle.silu(0.0) == 0.0
    for v in (0.25, 1.0, 3.5, 11.0, 40.0):
        assert oracle.silu(v) - oracle.silu(-v) == pytest.approx(v, rel=1e-14)          # silu(v) - silu(-v) = v
        assert oracle.silu(v) == pytest.approx(0.5 * v * (1.0 + np.tanh(0.5 * v)), rel=1e-13)   # the tanh form, library routine
    assert oracle.silu(40.0) == pytest.approx(40.0, rel=1e-15)
    assert abs(oracle.silu(-40.0)) < 1e-15
    # minimum of silu: its derivative vanishes where 1 + exp(-v) + v exp(-v) = 0, v = -1.2784645427610738
    v0 = -1.2784645427610738
    assert oracle.silu(v0) == pytest.approx(-0.2784645427610738, rel=1e-12)
    assert oracle.silu(v0 - 1e-3) > oracle.silu(v0) < oracle.silu(v0 + 1e-3)


def test_swiglu_is_silu_of_the_first_times_the_second():
    g = np.array([[0.0, 1.0, -2.0], [3.0, -0.5, 8.0]])
    u = np.array([[5.0, -2.0, 4.0], [0.5, 7.0, -1.0]])
    h = oracle.swiglu(g, u)
    want = np.array([[oracle.silu(a) * b for a, b in zip(rg, ru)] for rg, ru in zip(g, u)])
    assert np.array_equal(h, want)
    assert h[0, 0] == 0.0 and not np.array_equal(h, oracle.swiglu(u, g))            # a swapped operand shows


def test_bias_is_added_per_output_row():
    y = np.arange(6, dtype=np.float64).reshape(2, 3)
    b = np.array([0.5, -1.0, 2.0], dtype=np.float16).view(np.uint16)
    assert np.array_equal(oracle.add_bias(y, b), y + np.array([0.5, -1.0, 2.0]))
    assert np.array_equal(oracle.add_bias(y, np.zeros(3, dtype=np.uint16)), y)


# ---- data-free producer ---------------------------------------------------------------------------------------------
def test_rtn_codes_and_msb_planes_hand_worked():
    """A group whose values sit on 0, 1/255, .., 1: code = 255 * w exactly; planes are the binary digits of the code
    (Eq. 5), B_i = P_{7-K+i}: for K = 3 the planes are bits 5, 6, 7."""
    codes = np.array([0, 255, 0b10110101, 0b01100000, 0b00100000, 0b11100000, 7, 128] * 16, dtype=np.float64)
    w = (codes / 255.0)[None, :]
    z, lo, scale = producer.rtn_uint8(w, 128)
    assert np.array_equal(z[0], codes.astype(np.uint8)) and lo[0, 0] == 0.0 and scale[0, 0] == pytest.approx(1 / 255)
    b = producer.msb_planes(z, 3)
    assert b.shape == (3, 1, 128)
    assert b[:, 0, :8].T.tolist() == [[0, 0, 0], [1, 1, 1], [1, 0, 1], [1, 1, 0], [1, 0, 0], [1, 1, 1], [0, 0, 0], [0, 0, 1]]
    # Z = sum 2^i P_i
    assert np.array_equal(sum((producer.msb_planes(z, 8)[i].astype(np.int64) << i) for i in range(8)), z)


def test_rtn_rounds_to_nearest_ties_to_even_and_handles_constant_groups():
    w = np.zeros((1, 128))
    w[0, 1] = 255.0
    w[0, 2], w[0, 3], w[0, 4] = 0.5, 1.5, 2.49           # ties go to the even code
    z, _, _ = producer.rtn_uint8(w, 128)
    assert z[0, :5].tolist() == [0, 255, 0, 2, 2]
    z2, lo2, sc2 = producer.rtn_uint8(np.full((2, 64), 3.25), 64)
    assert not z2.any() and lo2[0, 0] == 3.25 and sc2[0, 0] == 1.0


@pytest.mark.parametrize("K", [2, 3])
def test_uniform_grid_is_recovered(K):
    """Proposition 1 turned round: weights that already lie on the uniform grid lo + s q, q in 0..2^K-1, come back with
    c0 = lo and c_i = s 2^(i-1), and the decode reproduces them."""
    rng = np.random.default_rng(K)
    out, g, ng = 6, 128, 2
    lo, s = -0.375, 2.0 ** -4
    q = rng.integers(0, 2 ** K, size=(out, g * ng))
    q[:, 0], q[:, 1] = 0, 2 ** K - 1                     # every group spans the grid
    q[:, g], q[:, g + 1] = 0, 2 ** K - 1
    w = lo + s * q
    bits, coef = producer.produce(w, K, g, alpha=0.0)
    assert np.array_equal(sum(bits[i].astype(np.int64) << i for i in range(K)), q)      # B_i carries binary digit i-1 of q
    cf = f16(coef).astype(np.float64)
    assert np.allclose(cf[0], lo, atol=1e-3) and all(np.allclose(cf[i], s * 2 ** (i - 1), rtol=2e-3) for i in range(1, K + 1))
    wq = f16(oracle.dequant(bits, coef, g)).astype(np.float64)
    assert np.max(np.abs(wq - w)) <= 2.0 ** -10


def test_fit_is_the_least_squares_solution():
    """Against the library's least-squares routine, and through the normal equations' defining property: the residual
    is orthogonal to every column of [1, b_1, .., b_K] (alpha = 0)."""
    rng = np.random.default_rng(11)
    out, g, K = 5, 64, 3
    w = rng.normal(0, 0.05, size=(out, 2 * g))
    z, _, _ = producer.rtn_uint8(w, g)
    bits = producer.msb_planes(z, K)
    c = producer.fit_coefficients(w, bits, g, alpha=0.0)
    for r in range(out):
        for G in range(2):
            cols = slice(G * g, (G + 1) * g)
            B = np.concatenate([np.ones((g, 1)), bits[:, r, cols].T], axis=1).astype(np.float64)
            ref = np.linalg.lstsq(B, w[r, cols], rcond=None)[0]
            assert np.allclose(c[:, r, G], ref, rtol=1e-8, atol=1e-10)
            assert np.allclose(B.T @ (B @ c[:, r, G] - w[r, cols]), 0.0, atol=1e-12)
    # a damped fit moves the coefficients, by little
    cd = producer.fit_coefficients(w, bits, g, alpha=1e-4)
    assert not np.array_equal(cd, c) and np.allclose(cd, c, rtol=5e-3, atol=1e-4)


def test_fit_survives_a_constant_plane():
    """A plane that is clear in the whole group makes the normal matrix singular; the damping keeps the system solvable
    and the fit of the remaining columns intact."""
    w = np.linspace(0.0, 0.4, 128)[None, :]              # codes 0..102 after the affine map? no: the map stretches to 0..255
    w[0, -1] = 10.0                                      # one outlier: every other code stays below 128, so the top plane is almost empty
    z, _, _ = producer.rtn_uint8(w, 128)
    bits = producer.msb_planes(z, 2)
    bits[1, 0, :] = 0                                    # force the most significant plane clear
    c = producer.fit_coefficients(w, bits, 128, alpha=1e-4)
    assert np.all(np.isfinite(c))


def test_more_planes_fit_better_and_structured_planes_beat_random_ones():
    rng = np.random.default_rng(2)
    w = rng.normal(0, 0.03, size=(8, 256))
    errs = []
    for K in (1, 2, 3, 4):
        bits, coef = producer.produce(w, K, 128)
        errs.append(np.mean((f16(oracle.dequant(bits, coef, 128)).astype(np.float64) - w) ** 2))
    assert errs[0] > errs[1] > errs[2] > errs[3]
    bits, coef = producer.produce(w, 2, 128)
    rnd = rng.integers(0, 2, size=bits.shape).astype(np.uint8)
    c_rnd = producer.fit_coefficients(w, rnd, 128).astype(np.float32).astype(np.float16).view(np.uint16)
    err_rnd = np.mean((f16(oracle.dequant(rnd, c_rnd, 128)).astype(np.float64) - w) ** 2)
    assert errs[1] < 0.5 * err_rnd


def test_truncated_view_keeps_the_top_planes_and_centres_the_dropped_ones():
    K, g = 3, 128
    bits = synth.plane_bits(5, 4, 256, K)
    coef = np.zeros((K + 1, 4, 2), dtype=np.float16)
    coef[0], coef[1], coef[2], coef[3] = -0.5, 0.125, 0.25, 0.5          # dyadic: every step exact
    coef = coef.view(np.uint16)
    b2, c2 = producer.truncate_planes(bits, coef, 2)
    assert np.array_equal(b2, bits[1:]) and c2.shape == (3, 4, 2)
    assert np.all(f16(c2[0]) == np.float16(-0.5 + 0.0625)) and np.array_equal(c2[1:], coef[2:])
    b1, c1 = producer.truncate_planes(bits, coef, 1)
    assert np.all(f16(c1[0]) == np.float16(-0.5 + 0.0625 + 0.125)) and np.array_equal(b1, bits[2:])
    # the view differs from the full decode by at most half the dropped coefficients
    w3 = f16(oracle.dequant(bits, coef, g)).astype(np.float64)
    w2 = f16(oracle.dequant(b2, c2, g)).astype(np.float64)
    assert np.max(np.abs(w3 - w2)) == 0.0625
    same = producer.truncate_planes(bits, coef, 3)
    assert np.array_equal(same[0], bits) and np.array_equal(same[1], coef)
