"""The few-token kernel (weights decoded in registers, warp-level tensor-core instructions) against the checker,
with the bound every linear kernel is held to."""
import numpy as np
import pytest

import oracle
from paper_2602_04163_b200 import binding, synth
from tests import gpu_util as G

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("K,g,out,in_,M", [
    (2, 128, 160, 640, 5),        # five 32-row groups, a ragged second slice (one block)
    (3, 128, 96, 384, 16),        # a single ragged slice (three blocks)
    (2, 128, 4096, 4096, 8),      # benchmark config 1 with eight tokens: several segments per CTA
    (3, 128, 1024, 2048, 13),
    (2, 256, 64, 1024, 3),        # a coefficient group every two blocks
    (1, 128, 32, 128, 1),
    (4, 128, 48, 1536, 9),        # sixteen candidates; 48 rows: the last row group holds 16 rows
    (2, 128, 272, 896, 17),       # two token tiles, the second holds one token
    (3, 128, 144, 512, 32),       # the most tokens this kernel takes
    (2, 128, 16, 128, 4),         # smallest supported shape
    (2, 64, 80, 384, 6),          # a coefficient group per half block (the paper's W2-G64)
    (3, 64, 272, 896, 24),        # W3-G64, two token tiles
    (4, 64, 48, 1536, 11),
    (1, 64, 1024, 2048, 2),
    (2, 128, 1040, 8192, 16),     # sixteen slices: four column ranges accumulate through the workspace
    (4, 128, 2064, 2048, 16),     # sixteen candidates with tasks of two row groups: several segments per CTA, ragged last task
    (4, 64, 1040, 4096, 20),      # the same with two token tiles and a coefficient group per half block
    (2, 256, 160, 640, 7),        # g = 256 with a short last group (the last slice holds one block of it)
    (3, 256, 272, 1152, 20),      # four and a half groups, two token tiles
])
def test_few_token_kernel(K, g, out, in_, M):
    h, bits, coef = G.make_layer(140 + K, out, in_, K, g, max_M=M)
    x = synth.activations(150 + K, M, in_)
    rows = None
    if out * in_ > 2 ** 22:
        rows = np.unique(np.concatenate([np.arange(0, out, 61), [15, 16, 31, 32, out - 17, out - 16, out - 1]]))
    G.check_linear(h, bits, coef, x, g, binding.KERNEL_FEW, rows=rows, what="few")
    # partial sums of different column ranges meet in binary32 atomic adds whose order is free: two calls may differ
    # by the last binary16 digit, no more (and workspace and counters must come back clean for the second call)
    y1 = G.run_linear(h, x, binding.KERNEL_FEW)
    y2 = G.run_linear(h, x, binding.KERNEL_FEW)
    assert np.allclose(y1, y2, rtol=2.0 ** -9, atol=1e-5)


@pytest.mark.parametrize("K", [1, 2, 3, 4])
def test_few_token_kernel_multiplies_the_dequantized_weights(K):
    """The operand is W^ itself: with one-hot tokens the kernel returns columns of bpdq_dequant exactly."""
    g, out, in_ = 128, 96, 640
    h, bits, coef = G.make_layer(7, out, in_, K, g, max_M=32)
    w = G.run_dequant(h).view(np.float16)
    for c0 in (0, 96, 608):
        x = np.zeros((32, in_), dtype=np.float16)
        x[np.arange(32), c0 + np.arange(32)] = 1.0
        y = G.run_linear(h, x.view(np.uint16), binding.KERNEL_FEW)
        assert np.array_equal(y.astype(np.float16), w[:, c0:c0 + 32].T)


@pytest.mark.parametrize("name,out,in_,K,M", [("gate", 29568, 8192, 2, 16), ("down", 8192, 29568, 3, 8), ("gate", 29568, 8192, 3, 32),
                                               ("down", 8192, 29568, 2, 5), ("7b_down", 3584, 18944, 2, 16), ("gate", 29568, 8192, 4, 12)])
def test_few_token_kernel_full_size_sampled(name, out, in_, K, M):
    """Benchmark-sized layers generated on the device; sampled rows against the checker."""
    g = 128
    h = binding.Handle(out, in_, K, g, None, 960 + K, M)
    x = synth.activations(961, M, in_)
    y = G.run_linear(h, x, binding.KERNEL_FEW)
    rows = np.unique(np.concatenate([np.arange(0, out, max(1, out // 40)), [0, 15, 16, 31, 32, out - 32, out - 16, out - 1]]))
    y_ref, a_ref = oracle.linear(synth.plane_bits(960 + K, out, in_, K, rows), synth.coefficients(960 + K, out, in_, K, g, rows), x, g)
    G.assert_linear_close(y[:, rows], y_ref, a_ref, name)
    assert np.all(np.isfinite(y))


def test_dispatcher_sends_3_to_16_tokens_to_the_few_token_kernel():
    K, g, out, in_ = 2, 128, 272, 896
    h, bits, coef = G.make_layer(171, out, in_, K, g, max_M=40)
    for M, same_as in ((2, binding.KERNEL_GEMV), (3, binding.KERNEL_FEW), (16, binding.KERNEL_FEW), (17, binding.KERNEL_GEMM)):
        x = synth.activations(172 + M, M, in_)
        G.check_linear(h, bits, coef, x, g, binding.KERNEL_AUTO, what=f"auto M={M}")
        n0 = h.bpdq_launch_count()
        ya = G.run_linear(h, x, binding.KERNEL_AUTO)
        assert h.bpdq_launch_count() == n0 + 1
        assert np.allclose(ya, G.run_linear(h, x, same_as), rtol=2.0 ** -9, atol=1e-5)
    h.bpdq_set_few_max_m(0)                                               # switched off: the tcgen05 kernel takes over
    x = synth.activations(180, 8, in_)
    assert np.array_equal(G.run_linear(h, x, binding.KERNEL_AUTO), G.run_linear(h, x, binding.KERNEL_GEMM))


def test_few_token_kernel_rejects_what_it_cannot_take():
    h, _, _ = G.make_layer(173, 32, 128, 2, 128, max_M=40)
    import torch
    x = torch.zeros((40, 128), dtype=torch.float16, device="cuda")
    y = torch.zeros((40, 32), dtype=torch.float16, device="cuda")
    n0 = h.bpdq_launch_count()
    with pytest.raises(binding.BpdqError) as ei:
        h.bpdq_linear_ex(x.data_ptr(), y.data_ptr(), binding.FEW_MAX_M + 1, binding.KERNEL_FEW, G.stream_ptr())
    assert ei.value.code == binding.ERR_INVALID and h.bpdq_launch_count() == n0


@pytest.mark.parametrize("g", [128, 64])
def test_dispatcher_with_sixteen_candidates(g):
    """K = 4 through bpdq_linear at the token counts either side of its thresholds (look-up-table kernel up to 3 tokens,
    2 at g = 64; few-token kernel to 16; tcgen05 beyond): every choice within the checker's bound."""
    K, out, in_ = 4, 272, 1536
    h, bits, coef = G.make_layer(190 + g, out, in_, K, g, max_M=20)
    for M in (1, 2, 3, 4, 16, 17):
        x = synth.activations(191 + M, M, in_)
        n0 = h.bpdq_launch_count()
        G.check_linear(h, bits, coef, x, g, binding.KERNEL_AUTO, what=f"K=4 g={g} M={M}")
        lut_max = 2 if g == 64 else 3
        passes = (M + 1) // 2 if M <= lut_max else 1      # the look-up-table kernel takes two tokens per pass
        assert h.bpdq_launch_count() - n0 == passes
    h.bpdq_destroy()
