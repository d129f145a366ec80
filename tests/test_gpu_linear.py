"""bpdq_linear (all kernels) against the checker: |y - y_ref| <= 4e-3 * sum|x w| + 1e-3 per element."""
import numpy as np
import pytest
import torch

import oracle
from paper_2602_04163_b200 import binding, synth
from tests import gpu_util as G

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("K,g,out,in_,M", [(2, 128, 160, 640, 1), (3, 128, 96, 384, 3), (1, 128, 32, 128, 1),
                                            (4, 128, 48, 256, 2), (2, 64, 80, 384, 1), (3, 256, 64, 768, 2)])
def test_simple_kernel(K, g, out, in_, M):
    h, bits, coef = G.make_layer(20 + K, out, in_, K, g, max_M=M)
    x = synth.activations(30 + K, M, in_)
    G.check_linear(h, bits, coef, x, g, binding.KERNEL_GEMV_SIMPLE, what="simple")


def test_m_zero_and_bad_arguments():
    import torch
    h, bits, coef = G.make_layer(1, 32, 128, 2, 128, max_M=2)
    h.bpdq_linear(0, 0, 0, G.stream_ptr())                              # M = 0: OK, nothing launched
    x = torch.zeros((2, 128), dtype=torch.float16, device="cuda")
    y = torch.zeros((2, 32), dtype=torch.float16, device="cuda")
    n0 = h.bpdq_launch_count()
    for args in ((x.data_ptr(), y.data_ptr(), 3), (x.data_ptr(), y.data_ptr(), -1), (0, y.data_ptr(), 1),
                 (x.data_ptr() + 2, y.data_ptr(), 1)):
        with pytest.raises(binding.BpdqError) as ei:
            h.bpdq_linear(*args, G.stream_ptr())
        assert ei.value.code == binding.ERR_INVALID
    with pytest.raises(binding.BpdqError):
        h.bpdq_linear_ex(x.data_ptr(), y.data_ptr(), 1, 99, G.stream_ptr())
    assert h.bpdq_launch_count() == n0                                   # no launch on rejected calls


@pytest.mark.parametrize("K,g,out,in_,M", [
    (2, 128, 160, 640, 1),       # 5 blocks: the second slice is ragged (1 block)
    (3, 128, 96, 384, 1),        # 3 blocks: a single ragged slice
    (2, 128, 4096, 4096, 1),     # benchmark config 1
    (3, 128, 1024, 2048, 2),
    (2, 256, 64, 1024, 3),
    (1, 128, 32, 128, 1),
    (4, 128, 48, 1536, 2),
    (2, 128, 272, 896, 4),       # 4 tokens = two passes of 2
    (3, 128, 144, 512, 7),       # 3 + 2 + 2
    (2, 128, 272, 896, 8),       # four passes
    (3, 128, 144, 1152, 16),     # the most tokens this kernel takes
    (2, 128, 16, 128, 1),        # smallest supported shape
    (2, 64, 80, 384, 1),         # a coefficient group per half block (the paper's W2-G64)
    (3, 64, 272, 896, 2),        # W3-G64, two tokens
    (4, 64, 48, 1536, 3),
    (1, 64, 1024, 2048, 1),
    (2, 256, 160, 640, 1),       # g = 256, two and a half groups: the last group is short (and so is the second slice)
    (3, 256, 272, 1152, 2),      # four and a half groups
])
def test_lut_kernel(K, g, out, in_, M):
    h, bits, coef = G.make_layer(40 + K, out, in_, K, g, max_M=M)
    x = synth.activations(50 + K, M, in_)
    rows = None
    if out * in_ > 2 ** 22:      # keep the checker's share to seconds: sampled rows, every tile boundary
        rows = np.unique(np.concatenate([np.arange(0, out, 61), [15, 16, 31, 32, out - 17, out - 16, out - 1]]))
    G.check_linear(h, bits, coef, x, g, binding.KERNEL_GEMV, rows=rows, what="lut")
    # slices are combined with binary32 atomic adds whose order is free: two calls may differ by
    # the last binary16 digit, no more (and the workspace must come back clean for the second call)
    y1 = G.run_linear(h, x, binding.KERNEL_GEMV)
    y2 = G.run_linear(h, x, binding.KERNEL_GEMV)
    assert np.allclose(y1, y2, rtol=2.0 ** -9, atol=1e-5)
    # the on-device cross-check kernel (rounded weights, sequential binary32 sum) is held to the checker's bound too
    G.check_linear(h, bits, coef, x, g, binding.KERNEL_GEMV_SIMPLE, rows=rows, what="simple")


def test_lut_kernel_special_inputs():
    """All-zero planes (y = sum_G c0 X_G), all-one planes, one-hot activations."""
    K, g, out, in_ = 2, 128, 64, 1024
    coef = synth.coefficients(8, out, in_, K, g)
    x = synth.activations(8, 1, in_)
    for fill in (0, 1):
        bits = np.full((K, out, in_), fill, dtype=np.uint8)
        h = binding.Handle(out, in_, K, g, binding.bpdq_pack(bits, coef, g), 0, 1)
        G.check_linear(h, bits, coef, x, g, binding.KERNEL_GEMV, what=f"fill{fill}")
    bits = synth.plane_bits(8, out, in_, K)
    h = binding.Handle(out, in_, K, g, binding.bpdq_pack(bits, coef, g), 0, 1)
    w = oracle.dequant(bits, coef, g).view(np.float16).astype(np.float64)
    for j in (0, 7, 8, 127, 128, 511, 512, 1023):
        xo = np.zeros((1, in_), dtype=np.float16)
        xo[0, j] = 1.0
        y = G.run_linear(h, xo.view(np.uint16), binding.KERNEL_GEMV)
        assert np.max(np.abs(y[0] - w[:, j])) <= 2.0 ** -10 * np.max(np.abs(w[:, j])) + 1e-6, j


@pytest.mark.parametrize("name,out,in_,K", [("gate", 29568, 8192, 2), ("down", 8192, 29568, 3), ("k", 1024, 8192, 2),
                                             ("7b_down", 3584, 18944, 2)])
def test_lut_kernel_full_size_sampled(name, out, in_, K):
    """Benchmark-sized layers generated on the device; sampled rows against the checker."""
    g = 128
    h = binding.Handle(out, in_, K, g, None, 900 + K, 1)
    x = synth.activations(901, 1, in_)
    y = G.run_linear(h, x, binding.KERNEL_GEMV)
    rows = np.unique(np.concatenate([np.arange(0, out, max(1, out // 40)), [0, 15, 16, out - 16, out - 1]]))
    y_ref, a_ref = oracle.linear(synth.plane_bits(900 + K, out, in_, K, rows),
                                 synth.coefficients(900 + K, out, in_, K, g, rows), x, g)
    G.assert_linear_close(y[:, rows], y_ref, a_ref, name)
    assert np.all(np.isfinite(y))


@pytest.mark.parametrize("M", [1, 2])
def test_chain_of_dependent_launches(M):
    """Three linears, each reading what the one before wrote, enqueued twice without a host wait in between, the
    second round on a different input written by a device-side copy that is itself still in flight.
    The look-up-table kernel starts before the kernel in front of it has finished (it only requests weights that
    early); every stage must still see the finished output of the stage before (a stale activation from the
    first round would show in the second), and the second round must find workspaces and counters as the first
    left them."""
    K, g = 2, 128
    dims = [(640, 384), (896, 640), (160, 896)]                     # (out, in): in of a stage is out of the one before
    layers = [G.make_layer(400 + k, o, i, K, g, max_M=M) for k, (o, i) in enumerate(dims)]
    inputs = [G.x_tensor(synth.activations(410 + rnd, M, dims[0][1])) for rnd in range(2)]
    x0 = torch.empty_like(inputs[0])
    ys = [torch.full((M, o), float("nan"), dtype=torch.float16, device="cuda") for o, _ in dims]
    sp = G.stream_ptr()
    for rnd in range(2):
        x0.copy_(inputs[rnd])                                        # same buffers in both rounds, new contents in the second
        src = x0
        for (h, _, _), y in zip(layers, ys):
            h.bpdq_linear_ex(src.data_ptr(), y.data_ptr(), M, binding.KERNEL_GEMV, sp)
            src = y
    torch.cuda.synchronize()
    src = inputs[1]                                                  # what is left is the second round's chain
    for k, ((h, bits, coef), y) in enumerate(zip(layers, ys)):
        h.bpdq_get_status(sp)
        x_bits = src.cpu().view(torch.int16).numpy().view(np.uint16)
        y_ref, a_ref = oracle.linear(bits, coef, x_bits, g)
        G.assert_linear_close(y.cpu().numpy().astype(np.float64), y_ref, a_ref, f"stage {k}")
        src = y
    assert not torch.equal(inputs[0], inputs[1])


def test_a_wait_that_runs_out_is_reported_and_leaves_the_handle_usable():
    """Every device-side wait of the library is bounded.  A barrier that nothing arrives at makes one run out: the status
    word then says BPDQ_ERR_TIMEOUT (once), the kernel ends by itself, and the same handle computes correctly afterwards."""
    h, bits, coef = G.make_layer(601, 160, 640, 2, 128, max_M=40)
    sp = G.stream_ptr()
    h.bpdq_get_status(sp)                                                # clean to begin with
    h.bpdq_probe_wait_limit(sp)
    with pytest.raises(binding.BpdqError) as ei:
        h.bpdq_get_status(sp)
    assert ei.value.code == binding.ERR_TIMEOUT
    h.bpdq_get_status(sp)                                                # reading the word cleared it
    for M, kernel in ((1, binding.KERNEL_GEMV), (5, binding.KERNEL_FEW), (40, binding.KERNEL_GEMM)):
        G.check_linear(h, bits, coef, synth.activations(602 + M, M, 640), 128, kernel, what=f"after the probe M={M}")
