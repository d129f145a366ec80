"""bpdq_linear_batch: several linears in one launch of the look-up-table kernel, against the checker."""
import numpy as np
import pytest
import torch

from paper_2602_04163_b200 import binding, synth
from tests import gpu_util as G

pytestmark = pytest.mark.gpu


def _run_batch(handles, xs_bits, M):
    xs = [G.x_tensor(x) for x in xs_bits]
    ys = [torch.full((M, h.out), float("nan"), dtype=torch.float16, device="cuda") for h in handles]
    binding.bpdq_linear_batch(handles, [x.data_ptr() for x in xs], [y.data_ptr() for y in ys], M, G.stream_ptr())
    torch.cuda.synchronize()
    for h in handles:
        h.bpdq_get_status(G.stream_ptr())
    return [y.cpu().numpy().astype(np.float64) for y in ys]


@pytest.mark.parametrize("K,M", [(2, 1), (3, 2), (2, 5), (1, 1), (3, 16), (1, 9)])
def test_batch_matches_checker_and_single_launches(K, M):
    import oracle
    g = 128
    shapes = [(160, 640), (48, 640), (272, 896), (16, 128), (1024, 2048)]     # ragged slices, tiny and multi-CTA linears
    layers = [G.make_layer(90 + k, o, i, K, g, max_M=M) for k, (o, i) in enumerate(shapes)]
    handles = [L[0] for L in layers]
    x640 = synth.activations(91, M, 640)
    xs = [x640, x640, synth.activations(92, M, 896), synth.activations(93, M, 128), synth.activations(94, M, 2048)]
    for rep in range(2):                                                      # the second call finds the workspaces as the first left them
        ys = _run_batch(handles, xs, M)
        for (h, bits, coef), x, y in zip(layers, xs, ys):
            y_ref, a_ref = oracle.linear(bits, coef, x, g)
            G.assert_linear_close(y, y_ref, a_ref, f"batch rep {rep} {h.out}x{h.in_}")
            y_single = G.run_linear(h, x, binding.KERNEL_AUTO)                # the same kernel as the batch takes for this M
            assert np.allclose(y, y_single, rtol=2.0 ** -9, atol=1e-5)


def test_batch_rejects_bad_arguments():
    h1, _, _ = G.make_layer(1, 32, 128, 2, 128, max_M=2)
    h2, _, _ = G.make_layer(2, 32, 128, 3, 128, max_M=2)
    x = torch.zeros((2, 128), dtype=torch.float16, device="cuda")
    y1 = torch.zeros((2, 32), dtype=torch.float16, device="cuda")
    y2 = torch.zeros((2, 32), dtype=torch.float16, device="cuda")
    n0 = h1.bpdq_launch_count()
    for handles, M in (([h1, h1], 1), ([h1, h2], 1), ([h1], 3), ([h1] * 0, 1)):
        with pytest.raises(binding.BpdqError) as ei:
            binding.bpdq_linear_batch(handles, [x.data_ptr()] * len(handles), [y1.data_ptr(), y2.data_ptr()][:len(handles)], M,
                                      G.stream_ptr())
        assert ei.value.code == binding.ERR_INVALID
    assert h1.bpdq_launch_count() == n0
    binding.bpdq_linear_batch([h1], [0], [0], 0, G.stream_ptr())              # M = 0: nothing to do


def test_batch_host_rejects_before_anything_is_enqueued():
    """The host-buffer call checks every rule of bpdq_linear_batch first: a rejected call launches nothing
    (not even the kernel that gathers the inputs)."""
    h1, _, _ = G.make_layer(1, 32, 128, 2, 128, max_M=2)
    h2, _, _ = G.make_layer(2, 32, 128, 3, 128, max_M=2)
    xh = torch.zeros((2, 128), dtype=torch.float16).pin_memory()
    yh = [torch.zeros((2, 32), dtype=torch.float16).pin_memory() for _ in range(2)]
    n0 = h1.bpdq_launch_count() + h2.bpdq_launch_count()
    for handles, M in (([h1, h1], 1), ([h1, h2], 1), ([h1], 3), ([h1], binding.GEMV_MAX_M + 1)):
        with pytest.raises(binding.BpdqError) as ei:
            binding.bpdq_linear_batch_host(handles, [xh.data_ptr()] * len(handles), [y.data_ptr() for y in yh][:len(handles)], M,
                                           G.stream_ptr())
        assert ei.value.code == binding.ERR_INVALID
    assert h1.bpdq_launch_count() + h2.bpdq_launch_count() == n0


@pytest.mark.parametrize("model,K", [("72b", 2), ("72b", 3), ("7b", 2)])
def test_batch_full_layer_sampled(model, K):
    """All seven linears of a Qwen2.5-shaped layer in one launch (the benchmark's step); sampled rows against the checker."""
    import oracle
    g = 128
    shapes = synth.QWEN25_72B_LAYER if model == "72b" else synth.QWEN25_7B_LAYER
    handles = [binding.Handle(o, i, K, g, None, 300 + li, 1) for li, (_, o, i) in enumerate(shapes)]
    xb = {i: synth.activations(301 + i, 1, i) for i in sorted({i for _, _, i in shapes})}
    ys = _run_batch(handles, [xb[i] for _, _, i in shapes], 1)
    for li, ((name, o, i), y) in enumerate(zip(shapes, ys)):
        rows = np.unique(np.concatenate([np.arange(0, o, max(1, o // 24)), [0, 15, 16, o - 16, o - 1]]))
        y_ref, a_ref = oracle.linear(synth.plane_bits(300 + li, o, i, K, rows), synth.coefficients(300 + li, o, i, K, g, rows), xb[i], g)
        G.assert_linear_close(y[:, rows], y_ref, a_ref, name)
        assert np.all(np.isfinite(y))
    for h in handles:
        h.bpdq_destroy()


@pytest.mark.parametrize("name,out,in_,K", [("gate", 29568, 8192, 2), ("gate", 29568, 8192, 3), ("down", 8192, 29568, 2),
                                             ("down", 8192, 29568, 3)])
def test_token_sweep_through_the_dispatcher(name, out, in_, K):
    """M = 1..64 on 72B-shaped projections through bpdq_linear (look-up-table kernel below the threshold,
    tensor-core kernel above); sampled rows against the checker."""
    import oracle
    g = 128
    h = binding.Handle(out, in_, K, g, None, 400 + K, 64)
    rows = np.unique(np.concatenate([np.arange(0, out, out // 12), [0, 127, 128, out - 1]]))
    bits, coef = synth.plane_bits(400 + K, out, in_, K, rows), synth.coefficients(400 + K, out, in_, K, g, rows)
    for M in (1, 2, 4, 8, 16, 32, 64):
        x = synth.activations(500 + M, M, in_)
        y = G.run_linear(h, x, binding.KERNEL_AUTO)
        y_ref, a_ref = oracle.linear(bits, coef, x, g)
        G.assert_linear_close(y[:, rows], y_ref, a_ref, f"{name} M={M}")
    h.bpdq_destroy()


def test_batch_host_buffers_match_device_call():
    K, g, M = 2, 128, 2
    shapes = [(160, 640), (48, 640), (272, 896)]
    layers = [G.make_layer(190 + k, o, i, K, g, max_M=M) for k, (o, i) in enumerate(shapes)]
    handles = [L[0] for L in layers]
    xs = [synth.activations(191 + k, M, i) for k, (_, i) in enumerate(shapes)]
    want = _run_batch(handles, xs, M)
    xh = [torch.from_numpy(x.view(np.int16).copy()).view(torch.float16).pin_memory() for x in xs]
    yh = [torch.full((M, o), float("nan"), dtype=torch.float16).pin_memory() for o, _ in shapes]
    binding.bpdq_linear_batch_host(handles, [x.data_ptr() for x in xh], [y.data_ptr() for y in yh], M, G.stream_ptr())
    for y, w in zip(yh, want):
        assert np.allclose(y.numpy().astype(np.float64), w, rtol=2.0 ** -9, atol=1e-5)


@pytest.mark.parametrize("pinned,M", [(True, 1), (True, 3), (False, 2)])
def test_batch_host_buffers_pinned_and_pageable(pinned, M):
    """Pinned buffers go through the gather launch with y stored straight into host memory (M = 3: two passes of the
    kernel); pageable ones through one copy per buffer.  Both must give what the device call gives."""
    K, g = 3, 128
    shapes = [(160, 640), (400, 1152)]
    layers = [G.make_layer(290 + k, o, i, K, g, max_M=M) for k, (o, i) in enumerate(shapes)]
    handles = [L[0] for L in layers]
    xs = [synth.activations(291 + k, M, i) for k, (_, i) in enumerate(shapes)]
    want = _run_batch(handles, xs, M)
    xh = [torch.from_numpy(x.view(np.int16).copy()).view(torch.float16) for x in xs]
    yh = [torch.full((M, o), float("nan"), dtype=torch.float16) for o, _ in shapes]
    if pinned:
        xh, yh = [x.pin_memory() for x in xh], [y.pin_memory() for y in yh]
    for _ in range(2):                                   # the second call finds the workspace as the first left it
        binding.bpdq_linear_batch_host(handles, [x.data_ptr() for x in xh], [y.data_ptr() for y in yh], M, G.stream_ptr())
        for y, w in zip(yh, want):
            assert np.allclose(y.numpy().astype(np.float64), w, rtol=2.0 ** -9, atol=1e-5)
            y.fill_(float("nan"))


@pytest.mark.parametrize("M", [1, 40])
def test_single_host_call(M):
    """bpdq_linear_host: one token takes the look-up-table kernel's host path, forty tokens the copies around the tensor-core kernel."""
    K, g, out, in_ = 2, 128, 272, 896
    h, bits, coef = G.make_layer(310, out, in_, K, g, max_M=M)
    x = synth.activations(311, M, in_)
    want = G.run_linear(h, x, binding.KERNEL_AUTO)
    xh = torch.from_numpy(x.view(np.int16).copy()).view(torch.float16).pin_memory()
    yh = torch.full((M, out), float("nan"), dtype=torch.float16).pin_memory()
    h.bpdq_linear_host(xh.data_ptr(), yh.data_ptr(), M, G.stream_ptr())
    assert np.allclose(yh.numpy().astype(np.float64), want.astype(np.float64), rtol=2.0 ** -9, atol=1e-5)
