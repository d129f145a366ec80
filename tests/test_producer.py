"""The library's host-side producers against the checker's (oracle/producer.py): planes bit-exact, coefficients equal
after the binary16 rounding up to one last digit (both solve the same normal equations in binary64, by different
routes), the truncated view bit-exact.  CPU only."""
import numpy as np
import pytest

import oracle
from oracle import producer
from paper_2602_04163_b200 import binding


def _weights(seed, out, in_):
    rng = np.random.default_rng(seed)
    w = rng.normal(0.0, 0.02, size=(out, in_)) * (1.0 + 4.0 * (rng.random((out, 1)) < 0.1))     # a few rows of larger scale
    w[rng.random(w.shape) < 0.002] *= 12.0                                                       # outliers, as trained weights have
    return w.astype(np.float32)


@pytest.mark.parametrize("K,g,out,in_", [(2, 128, 32, 512), (3, 64, 16, 256), (4, 128, 16, 384), (1, 256, 16, 512)])
def test_datafree_producer_matches_the_checker(K, g, out, in_):
    w = _weights(K, out, in_)
    bits, coef = binding.bpdq_quantize_datafree(w, K, g)
    bits_ref, coef_ref = producer.produce(w.astype(np.float64), K, g)
    assert np.array_equal(bits, bits_ref)
    a, b = coef.view(np.float16).astype(np.float64), coef_ref.view(np.float16).astype(np.float64)
    assert np.all(np.abs(a - b) <= 2.0 ** -10 * np.abs(b) + 2.0 ** -24)
    assert np.mean(coef == coef_ref) > 0.98
    # and the reconstruction error is what the checker's tensors give
    e = np.mean((oracle.dequant(bits, coef, g).view(np.float16).astype(np.float64) - w) ** 2)
    e_ref = np.mean((oracle.dequant(bits_ref, coef_ref, g).view(np.float16).astype(np.float64) - w) ** 2)
    assert e == pytest.approx(e_ref, rel=1e-3) and e < np.mean(w.astype(np.float64) ** 2) * (0.5 if K == 1 else 0.2)


def test_datafree_producer_constant_group_and_bad_arguments():
    w = np.full((16, 128), 0.125, dtype=np.float32)
    bits, coef = binding.bpdq_quantize_datafree(w, 2, 128)
    assert not bits.any()
    assert np.all(oracle.dequant(bits, coef, 128).view(np.float16) == np.float16(0.125))
    w[3, 5] = np.nan
    with pytest.raises(binding.BpdqError) as ei:
        binding.bpdq_quantize_datafree(w, 2, 128)
    assert ei.value.code == binding.ERR_INVALID
    with pytest.raises(binding.BpdqError):
        binding.bpdq_quantize_datafree(np.zeros((10, 128), dtype=np.float32), 2, 128)     # out % 16 != 0


@pytest.mark.parametrize("K,K2", [(3, 2), (3, 1), (4, 2), (2, 2)])
def test_truncated_view_matches_the_checker(K, K2):
    g, out, in_ = 128, 32, 512
    w = _weights(10 + K, out, in_)
    bits, coef = binding.bpdq_quantize_datafree(w, K, g)
    b2, c2 = binding.bpdq_truncate_planes(bits, coef, g, K2)
    rb, rc = producer.truncate_planes(bits, coef, K2)
    assert np.array_equal(b2, rb) and np.array_equal(c2, rc)
    # it is a valid tensor of K2 planes: it packs, and fewer planes cost accuracy
    assert binding.bpdq_pack(b2, c2, g).size == binding.bpdq_packed_bytes(out, in_, K2, g)
    if K2 < K:
        e_full = np.mean((oracle.dequant(bits, coef, g).view(np.float16).astype(np.float64) - w) ** 2)
        e_view = np.mean((oracle.dequant(b2, c2, g).view(np.float16).astype(np.float64) - w) ** 2)
        assert e_view > e_full
