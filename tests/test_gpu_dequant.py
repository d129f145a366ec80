"""bpdq_dequant and the device-side weight generator against the checker: bit-exact."""
import numpy as np
import pytest

import oracle
from paper_2602_04163_b200 import binding, synth
from tests import gpu_util as G

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("K,g,out,in_", [(2, 128, 160, 640), (3, 128, 96, 384), (1, 128, 32, 128),
                                          (4, 128, 48, 256), (2, 64, 80, 384), (3, 256, 64, 768), (2, 128, 16, 128),
                                          (2, 256, 160, 640), (3, 256, 272, 1152)])   # g = 256 with a short last group (2.5 and 4.5 groups)
def test_dequant_bit_exact(K, g, out, in_):
    h, bits, coef = G.make_layer(10 + K, out, in_, K, g)
    w = G.run_dequant(h)
    assert np.array_equal(w, oracle.dequant(bits, coef, g))


def test_dequant_adversarial_coefficients():
    """Raw binary16 patterns: subnormals, large values that overflow, negative zero offsets, NaN-free."""
    K, g, out, in_ = 3, 128, 64, 256
    rng = np.random.default_rng(5)
    bits = synth.plane_bits(2, out, in_, K)
    coef = rng.integers(0, 0x7C00, size=(K + 1, out, in_ // g)).astype(np.uint16)
    coef ^= (rng.integers(0, 2, size=coef.shape).astype(np.uint16) << 15)
    coef[0, :8, 0] = 0x8000                                    # -0.0 offsets
    coef[:, 8, 0] = [np.float16(2048).view(np.uint16), np.float16(1).view(np.uint16),
                     np.float16(2.0 ** -13).view(np.uint16), np.float16(2.0 ** -13).view(np.uint16)]  # order of adds
    h = binding.Handle(out, in_, K, g, binding.bpdq_pack(bits, coef, g), 0, 1)
    assert np.array_equal(G.run_dequant(h), oracle.dequant(bits, coef, g))


@pytest.mark.parametrize("K,g,in_", [(2, 128, 512), (3, 128, 512), (4, 64, 512), (2, 256, 640)])
def test_device_generator_matches_host_generator(K, g, in_):
    out = 96
    h = binding.Handle(out, in_, K, g, None, 77, 1)
    blob = h.bpdq_read_blob()
    bits, coef = oracle.unpack(blob, out, in_, K, g)
    assert np.array_equal(bits, synth.plane_bits(77, out, in_, K))
    assert np.array_equal(coef, synth.coefficients(77, out, in_, K, g))
    assert np.array_equal(blob, binding.bpdq_pack(bits, coef, g))


def test_dequant_full_size_sampled_rows():
    """72B-shaped gate (29568 x 8192, K=3), generated on the device; sampled rows against the checker."""
    out, in_, K, g = 29568, 8192, 3, 128
    h = binding.Handle(out, in_, K, g, None, 123, 1)
    w = G.run_dequant(h)
    rows = np.array([0, 1, 15, 16, 31, 4097, 12345, 29552, 29567])
    want = oracle.dequant(synth.plane_bits(123, out, in_, K, rows), synth.coefficients(123, out, in_, K, g, rows), g)
    assert np.array_equal(w[rows], want)
    # property at full size: at most 2^K distinct values per (row, group) on a strided sample of rows
    sample = w[::997].reshape(-1, in_ // g, g)
    assert max(len(np.unique(grp)) for row in sample for grp in row) <= 2 ** K
