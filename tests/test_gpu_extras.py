"""Steps around the linear map on the GPU against the checker: input-channel permutation, bias, the gated unit of a
(gate, up) pair, and weights made by the data-free producer (structured planes instead of random ones)."""
import numpy as np
import pytest
import torch

import oracle
from oracle import producer
from paper_2602_04163_b200 import binding, synth
from tests import gpu_util as G

pytestmark = pytest.mark.gpu

KERNELS = [("lut", binding.KERNEL_GEMV, 1), ("lut", binding.KERNEL_GEMV, 2), ("few", binding.KERNEL_FEW, 5), ("few", binding.KERNEL_FEW, 20),
           ("tile", binding.KERNEL_GEMM, 40), ("persistent", binding.KERNEL_GEMM, 300), ("simple", binding.KERNEL_GEMV_SIMPLE, 3),
           ("auto", binding.KERNEL_AUTO, 9)]


def _group_perm(in_, g, seed):
    rng = np.random.default_rng(seed)
    return np.concatenate([G_ * g + rng.permutation(g) for G_ in rng.permutation(in_ // g)]).astype(np.int32)


@pytest.mark.parametrize("name,kernel,M", KERNELS)
def test_permutation_in_every_kernel(name, kernel, M):
    K, g, out, in_ = 3, 128, 272, 896
    h, bits, coef = G.make_layer(501, out, in_, K, g, max_M=M)
    x = synth.activations(502 + M, M, in_)
    perm = _group_perm(in_, g, 503)
    h.bpdq_set_input_permutation(perm)
    y = G.run_linear(h, x, kernel)
    y_ref, a_ref = oracle.linear_perm(bits, coef, x, perm.astype(np.int64), g)
    G.assert_linear_close(y, y_ref, a_ref, f"perm {name}")
    y_plain, _ = oracle.linear(bits, coef, x, g)
    assert np.max(np.abs(y_ref - y_plain)) > 0.1                       # the permutation matters for this input
    h.bpdq_set_input_permutation(None)                                   # and can be taken away again
    G.check_linear(h, bits, coef, x, g, kernel, what=f"identity {name}")


def test_permutation_rejects_what_is_not_one_and_works_in_a_batch():
    K, g, M = 2, 128, 6
    shapes = [(160, 640), (48, 640)]
    layers = [G.make_layer(510 + k, o, i, K, g, max_M=M) for k, (o, i) in enumerate(shapes)]
    bad = np.arange(640, dtype=np.int32)
    bad[3] = 4
    with pytest.raises(binding.BpdqError) as ei:
        layers[0][0].bpdq_set_input_permutation(bad)
    assert ei.value.code == binding.ERR_INVALID
    perm = _group_perm(640, g, 511)
    layers[1][0].bpdq_set_input_permutation(perm)                        # one linear of the batch is permuted, the other is not
    for Mb in (1, M):                                                    # look-up-table launch, few-token launch
        x = synth.activations(512 + Mb, Mb, 640)
        xt = G.x_tensor(x)
        ys = [torch.full((Mb, o), float("nan"), dtype=torch.float16, device="cuda") for o, _ in shapes]
        binding.bpdq_linear_batch([L[0] for L in layers], [xt.data_ptr()] * 2, [y.data_ptr() for y in ys], Mb, G.stream_ptr())
        torch.cuda.synchronize()
        y0, a0 = oracle.linear(layers[0][1], layers[0][2], x, g)
        y1, a1 = oracle.linear_perm(layers[1][1], layers[1][2], x, perm.astype(np.int64), g)
        G.assert_linear_close(ys[0].cpu().numpy().astype(np.float64), y0, a0, f"batch plain M={Mb}")
        G.assert_linear_close(ys[1].cpu().numpy().astype(np.float64), y1, a1, f"batch perm M={Mb}")


@pytest.mark.parametrize("name,kernel,M", KERNELS + [("split", binding.KERNEL_GEMM, 24)])
def test_bias_in_every_kernel(name, kernel, M):
    K, g = 2, 128
    out, in_ = (256, 4096) if name == "split" else (272, 896)           # few row tiles and long rows: the tile kernel splits the input dimension
    h, bits, coef = G.make_layer(520, out, in_, K, g, max_M=M)
    x = synth.activations(521 + M, M, in_)
    bias = (np.random.default_rng(522).normal(0, 0.5, out)).astype(np.float16)
    h.bpdq_set_bias(bias.view(np.uint16))
    y = G.run_linear(h, x, kernel)
    y_ref, a_ref = oracle.linear(bits, coef, x, g)
    want = oracle.add_bias(y_ref, bias.view(np.uint16))
    err = np.abs(y - want)
    bound = G.TOL_REL * (a_ref + np.abs(bias.astype(np.float64))[None, :]) + G.TOL_ABS   # the rounded value may now be as large as a + |b|
    assert np.all(err <= bound), f"bias {name}: max err/bound {np.max(err / bound):.3g}"
    assert np.max(np.abs(want - y_ref)) > 0.5
    h.bpdq_set_bias(None)
    G.check_linear(h, bits, coef, x, g, kernel, what=f"no bias {name}")


@pytest.mark.parametrize("M,with_bias,with_perm", [(1, False, False), (2, True, True), (8, False, False), (16, True, True), (40, True, False),
                                                    (300, False, True)])
def test_gated_unit_of_a_gate_up_pair(M, with_bias, with_perm):
    """h = silu(x Wg^T) * (x Wu^T): one launch up to the few-token threshold, three above; twice in a row (the second
    call finds workspaces and counters as the first left them)."""
    K, g, out, in_ = 2, 128, 400, 1152
    hg, bg, cg = G.make_layer(530, out, in_, K, g, max_M=M)
    hu, bu, cu = G.make_layer(531, out, in_, K, g, max_M=M)
    x = synth.activations(532 + M, M, in_)
    gy, ga = oracle.linear(bg, cg, x, g)
    uy, ua = oracle.linear(bu, cu, x, g)
    if with_perm:
        perm = _group_perm(in_, g, 533)
        hg.bpdq_set_input_permutation(perm)
        hu.bpdq_set_input_permutation(perm)
        gy, ga = oracle.linear_perm(bg, cg, x, perm.astype(np.int64), g)
        uy, ua = oracle.linear_perm(bu, cu, x, perm.astype(np.int64), g)
    if with_bias:
        b1 = np.random.default_rng(534).normal(0, 0.3, out).astype(np.float16)
        b2 = np.random.default_rng(535).normal(0, 0.3, out).astype(np.float16)
        hg.bpdq_set_bias(b1.view(np.uint16))
        hu.bpdq_set_bias(b2.view(np.uint16))
        gy, uy = oracle.add_bias(gy, b1.view(np.uint16)), oracle.add_bias(uy, b2.view(np.uint16))
        ga, ua = ga + np.abs(b1.astype(np.float64)), ua + np.abs(b2.astype(np.float64))
    want = oracle.swiglu(gy, uy)
    # first-order propagation of the two linears' accepted errors through the unit (|silu'| <= 1.1), plus the output's rounding
    dg, du = G.TOL_REL * ga + G.TOL_ABS, G.TOL_REL * ua + G.TOL_ABS
    silu_g = oracle.swiglu(gy, np.ones_like(gy))
    bound = 1.1 * (np.abs(uy) + du) * dg + (np.abs(silu_g) + 1.1 * dg) * du + 2.0 ** -10 * np.abs(want) + 1e-4
    xt = G.x_tensor(x)
    n0 = hg.bpdq_launch_count() + hu.bpdq_launch_count()
    for rep in range(2):
        hout = torch.full((M, out), float("nan"), dtype=torch.float16, device="cuda")
        binding.bpdq_gate_up_swiglu(hg, hu, xt.data_ptr(), hout.data_ptr(), M, G.stream_ptr())
        torch.cuda.synchronize()
        hg.bpdq_get_status(G.stream_ptr())
        err = np.abs(hout.cpu().numpy().astype(np.float64) - want)
        assert np.all(err <= bound), f"rep {rep}: max err/bound {np.nanmax(err / bound):.3g}"
    fused = M <= 16
    if fused and not (with_perm and M > 2):
        assert hg.bpdq_launch_count() + hu.bpdq_launch_count() == n0 + 2          # one launch per call
    # the two handles still work on their own afterwards
    hg.bpdq_set_input_permutation(None); hg.bpdq_set_bias(None)
    G.check_linear(hg, bg, cg, x, g, what="gate alone afterwards")


def test_gated_unit_rejects_mismatched_pairs():
    h1, _, _ = G.make_layer(540, 64, 256, 2, 128, max_M=2)
    h2, _, _ = G.make_layer(541, 48, 256, 2, 128, max_M=2)
    x = torch.zeros((2, 256), dtype=torch.float16, device="cuda")
    y = torch.zeros((2, 64), dtype=torch.float16, device="cuda")
    for a, b, M in ((h1, h2, 1), (h1, h1, 1), (h1, h2, 3)):
        with pytest.raises(binding.BpdqError) as ei:
            binding.bpdq_gate_up_swiglu(a, b, x.data_ptr(), y.data_ptr(), M, G.stream_ptr())
        assert ei.value.code == binding.ERR_INVALID


@pytest.mark.parametrize("K,g", [(2, 128), (3, 64), (4, 128)])
def test_data_free_weights_through_every_kernel(K, g):
    """Planes that are the most significant bits of real-valued weights (Eq. 5) with fitted coefficients (Eq. 6,
    U_loc = I), not random ones: dequant bit-exact, linears within the bound, and the truncated view served as a
    layer of its own."""
    out, in_ = 272, 1152
    rng = np.random.default_rng(550 + K)
    w = rng.normal(0, 0.02, size=(out, in_)).astype(np.float32)
    w[rng.random(w.shape) < 0.002] *= 10.0
    bits, coef = binding.bpdq_quantize_datafree(w, K, g)
    rb, rc = producer.produce(w.astype(np.float64), K, g)
    assert np.array_equal(bits, rb)
    for tag, (b_, c_, K_) in {"full": (bits, coef, K), "view": (*binding.bpdq_truncate_planes(bits, coef, g, max(1, K - 1)), max(1, K - 1))}.items():
        h = binding.Handle(out, in_, K_, g, binding.bpdq_pack(b_, c_, g), 0, 300)
        assert np.array_equal(G.run_dequant(h), oracle.dequant(b_, c_, g)), tag
        for M, kernel in ((1, binding.KERNEL_GEMV), (7, binding.KERNEL_FEW), (40, binding.KERNEL_GEMM), (300, binding.KERNEL_GEMM)):
            G.check_linear(h, b_, c_, synth.activations(560 + M, M, in_), g, kernel, what=f"{tag} M={M}")
        h.bpdq_destroy()
    # the quantized layer approximates the original one: output error well below the output's own scale
    x = synth.activations(570, 4, in_)
    y_q, _ = oracle.linear(bits, coef, x, g)
    y_w = x.view(np.float16).astype(np.float64) @ w.astype(np.float64).T
    assert np.sqrt(np.mean((y_q - y_w) ** 2)) < (0.45, 0.45, 0.25, 0.13)[K - 1] * np.sqrt(np.mean(y_w ** 2))
