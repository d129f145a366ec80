"""A decoder layer's launches recorded once into a CUDA graph and replayed: the calls of the C ABI enqueue kernels on the
caller's stream and nothing else once a handle has been used (no allocation, no host wait), so a stream capture
takes them as they are.  The replayed graph must give what the direct calls give, for new activations written into
the same buffers, with each of the three kernel families (look-up-table, few-token, tcgen05)."""
import numpy as np
import pytest
import torch

import oracle
from paper_2602_04163_b200 import binding, synth
from tests import gpu_util as G

pytestmark = pytest.mark.gpu

# a small decoder layer: q k v o gate up down (out, in); hidden 512, kv 128, intermediate 1408
LAYER = [("q", 512, 512), ("k", 128, 512), ("v", 128, 512), ("o", 512, 512), ("gate", 1408, 512), ("up", 1408, 512), ("down", 512, 1408)]


def _enqueue_layer(hs, x_hidden, x_inter, ys, h_unit, w_q, M, sp):
    """The launches a decoder issues for its seven projections: {q, k, v}, {o}, the gated unit over {gate, up}, {down}.
    (Attention and the residual adds are not part of this library: o and down read given activations.)"""
    if M <= binding.GEMV_MAX_M:
        binding.bpdq_linear_batch(hs[0:3], [x_hidden.data_ptr()] * 3, [y.data_ptr() for y in ys[0:3]], M, sp)
    else:
        for k in range(3):
            hs[k].bpdq_linear(x_hidden.data_ptr(), ys[k].data_ptr(), M, sp)
    hs[3].bpdq_linear(x_hidden.data_ptr(), ys[3].data_ptr(), M, sp)
    binding.bpdq_gate_up_swiglu(hs[4], hs[5], x_hidden.data_ptr(), h_unit.data_ptr(), M, sp)
    hs[6].bpdq_linear(x_inter.data_ptr(), ys[6].data_ptr(), M, sp)
    hs[0].bpdq_dequant(w_q.data_ptr(), sp)               # not a decoder's step; recorded to show that it can be


@pytest.mark.parametrize("K,M", [(2, 1), (3, 2), (2, 8), (3, 40), (2, 300)])
def test_decoder_layer_as_a_cuda_graph(K, M):
    g = 128
    layers = [G.make_layer(800 + li, o, i, K, g, max_M=M) for li, (_, o, i) in enumerate(LAYER)]
    hs = [L[0] for L in layers]
    stream = torch.cuda.Stream()
    sp = stream.cuda_stream
    x_hidden = torch.zeros((M, 512), dtype=torch.float16, device="cuda")
    x_inter = torch.zeros((M, 1408), dtype=torch.float16, device="cuda")
    ys = [torch.zeros((M, o), dtype=torch.float16, device="cuda") for _, o, _ in LAYER]
    h_unit = torch.zeros((M, 1408), dtype=torch.float16, device="cuda")
    w_q = torch.zeros((512, 512), dtype=torch.float16, device="cuda")

    def load(seed):
        xh, xi = synth.activations(seed, M, 512), synth.activations(seed + 1, M, 1408)
        x_hidden.copy_(G.x_tensor(xh))
        x_inter.copy_(G.x_tensor(xi))
        return xh, xi

    # first use outside the capture: shared-memory opt-ins, launch plans and tensor maps are set up once per handle
    load(810)
    with torch.cuda.stream(stream):
        _enqueue_layer(hs, x_hidden, x_inter, ys, h_unit, w_q, M, sp)
    stream.synchronize()

    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph, stream=stream):
        _enqueue_layer(hs, x_hidden, x_inter, ys, h_unit, w_q, M, sp)

    for seed in (820, 830):                              # two replays, each on new activations in the captured buffers
        xh, xi = load(seed)
        for y in ys:
            y.fill_(float("nan"))
        h_unit.fill_(float("nan"))
        w_q.zero_()
        torch.cuda.synchronize()
        graph.replay()
        torch.cuda.synchronize()
        for h in hs:
            h.bpdq_get_status(G.stream_ptr())
        for li, (name, o, i) in enumerate(LAYER):
            if name in ("gate", "up"):
                continue
            x = xi if name == "down" else xh
            y_ref, a_ref = oracle.linear(layers[li][1], layers[li][2], x, g)
            G.assert_linear_close(ys[li].cpu().numpy().astype(np.float64), y_ref, a_ref, f"replayed {name} seed {seed}")
        yg, ag = oracle.linear(layers[4][1], layers[4][2], xh, g)
        yu, au = oracle.linear(layers[5][1], layers[5][2], xh, g)
        h_ref = oracle.swiglu(yg, yu)
        got = h_unit.cpu().numpy().astype(np.float64)
        # the unit's bound: first-order propagation of the two linears' bounds (|silu'| <= 1.1) plus the last rounding
        dg, du = G.TOL_REL * ag + G.TOL_ABS, G.TOL_REL * au + G.TOL_ABS
        silu_g = oracle.swiglu(yg, np.ones_like(yg))
        bound = 1.1 * (np.abs(yu) + du) * dg + (np.abs(silu_g) + 1.1 * dg) * du + 2.0 ** -10 * np.abs(h_ref) + 1e-4
        assert np.all(np.abs(got - h_ref) <= bound), f"replayed gated unit seed {seed}"
        assert np.array_equal(w_q.view(torch.int16).cpu().numpy().view(np.uint16), oracle.dequant(layers[0][1], layers[0][2], g))
    for h in hs:
        h.bpdq_destroy()
