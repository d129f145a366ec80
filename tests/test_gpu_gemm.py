"""bpdq_gemm (TMA + tcgen05 tensor-core kernel) against the checker, same bound as every linear kernel."""
import numpy as np
import pytest

import oracle
from paper_2602_04163_b200 import binding, synth
from tests import gpu_util as G

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("K,g,out,in_,M", [
    (2, 128, 128, 128, 16),      # one tile, one 128-column block, two stages
    (2, 128, 128, 1024, 32),     # more k-blocks than pipeline stages: every barrier wraps
    (3, 128, 256, 512, 33),      # token tile of 64 with a ragged tail
    (1, 128, 128, 256, 5),
    (2, 64, 128, 384, 64),       # a coefficient group per k-block
    (3, 256, 256, 768, 100),     # a coefficient group every four k-blocks, token tile 128
    (2, 128, 160, 640, 130),     # ragged last row tile (160 = 128 + 32), token tile 256 with a ragged tail
    (3, 128, 384, 2048, 257),    # two token tiles of 256, the second holds one token
    (2, 128, 1024, 1024, 300),
    (2, 128, 128, 128, 1),       # a single token through the tensor-core path
    (4, 128, 256, 512, 40),      # sixteen candidates per group (the paper's W4-G128): two byte-permutes and a select
    (4, 64, 128, 384, 300),
    (2, 128, 256, 4096, 40),     # few row tiles, long rows: four CTAs share an output tile (split over the input dimension)
    (3, 64, 128, 8192, 64),      # eight-way split
    (4, 128, 384, 2048, 7),      # two-way split, ragged token tile
    (2, 128, 256, 4096, 100),    # 128-token tile shared by four CTAs (split over the input dimension), two CTAs per SM
    (3, 128, 384, 2048, 128),    # 128-token tile, two-way split, all 128 token columns in use
    (2, 256, 160, 640, 24),      # g = 256 with a short last group: tile kernel
    (3, 256, 272, 1152, 200),    # ... 256-token kernel
    (2, 256, 160, 1664, 600),    # ... 512-token kernel (six and a half groups)
    (2, 128, 256, 384, 20500),   # 162 output tiles for 148 persistent CTAs: a second tile per CTA, odd number of blocks per tile
    (4, 128, 128, 640, 38000),   # 149 tiles, three-stage ring (K = 4), odd number of blocks per tile
    (3, 64, 160, 640, 24),       # tile kernel, ragged last row tile (the tensor maps fill the missing rows), two groups per block
    (1, 256, 144, 1024, 100),    # tile kernel with the 128-token tile, ragged row tile, a group every two blocks
    (2, 128, 400, 1152, 9),      # 16-token tile, odd number of blocks, rings wrap at different stages
    (2, 128, 256, 512, 256),     # the most tokens the 256-token kernel takes
    (3, 128, 384, 2048, 200),    # 256-token kernel, ragged token tile
    (2, 64, 160, 640, 700),      # 512-token kernel: two token tiles (the second holds 188), ragged row tile, a group per half block
    (3, 256, 272, 1024, 513),    # 512-token kernel: the second token tile holds one token; a group every two blocks
    (1, 128, 128, 256, 1030),    # 512-token kernel: two blocks per tile, three token tiles
    (4, 128, 256, 384, 300),     # 512-token kernel with sixteen candidates (largest packed blocks), odd number of blocks per tile
])
def test_gemm_kernel(K, g, out, in_, M):
    h, bits, coef = G.make_layer(60 + K, out, in_, K, g, max_M=M)
    x = synth.activations(70 + K, M, in_)
    rows = None
    if M > 4096:                 # many tokens: every token, rows sampled from every 32-row quadrant of every row tile
        rows = np.unique(np.concatenate([np.arange(0, out, 37), [0, 31, 32, 127, out - 128, out - 1]]))
    G.check_linear(h, bits, coef, x, g, binding.KERNEL_GEMM, rows=rows, what="gemm")
    y1 = G.run_linear(h, x, binding.KERNEL_GEMM)
    y2 = G.run_linear(h, x, binding.KERNEL_GEMM)
    if M > 128 or in_ < 2048:
        assert np.array_equal(y1, y2)                    # one CTA per output tile, fixed accumulation order: bit-identical reruns
    else:                                                # CTAs that share a tile add their parts in a free order: last binary16 digit
        assert np.allclose(y1, y2, rtol=2.0 ** -9, atol=1e-5)


@pytest.mark.parametrize("K", [1, 2, 3, 4])
def test_gemm_equals_dequant_times_x(K):
    """The decoded operand is W^ itself: with one-hot tokens the kernel must return columns of bpdq_dequant exactly."""
    g, out, in_ = 128, 256, 512
    h, bits, coef = G.make_layer(5, out, in_, K, g, max_M=in_)
    w = G.run_dequant(h).view(np.float16)
    x = np.eye(in_, dtype=np.float16)                    # token t selects column t
    y = G.run_linear(h, x.view(np.uint16), binding.KERNEL_GEMM)
    assert np.array_equal(y.astype(np.float16), w.T)


def test_dispatch_sends_large_m_to_the_tensor_core_kernel():
    K, g, out, in_, M = 2, 128, 256, 512, 48
    h, bits, coef = G.make_layer(9, out, in_, K, g, max_M=M)
    x = synth.activations(10, M, in_)
    G.check_linear(h, bits, coef, x, g, binding.KERNEL_AUTO, what="auto")
    assert np.array_equal(G.run_linear(h, x, binding.KERNEL_AUTO), G.run_linear(h, x, binding.KERNEL_GEMM))


@pytest.mark.parametrize("name,out,in_,K,M", [("gate", 29568, 8192, 3, 2048), ("down", 8192, 29568, 2, 512)])
def test_gemm_full_size_sampled(name, out, in_, K, M):
    """72B-shaped layers generated on the device; a row of every few tiles, every token, against the checker."""
    g = 128
    h = binding.Handle(out, in_, K, g, None, 950 + K, M)
    x = synth.activations(951, M, in_)
    y = G.run_linear(h, x, binding.KERNEL_GEMM)
    rows = np.unique(np.concatenate([np.arange(0, out, 997), [0, 127, 128, out - 129, out - 128, out - 1]]))
    y_ref, a_ref = oracle.linear(synth.plane_bits(950 + K, out, in_, K, rows),
                                 synth.coefficients(950 + K, out, in_, K, g, rows), x, g)
    G.assert_linear_close(y[:, rows], y_ref, a_ref, name)
    assert np.all(np.isfinite(y))
