"""The two largest benchmark workloads against the checker, with the benchmark's own seeds and launch shapes:
the 80-layer decode sweep (20.8 GB of packed weights generated on the device, one token through each of the 560
linears, once as 560 bpdq_linear calls and once as 80 bpdq_linear_batch calls) and the prefill pass of one
72B-shaped layer at K = 3 with 8192 tokens.  The checker cannot redo these sizes in full, so it recomputes sampled
outputs one by one: for the sweep a handful of rows of every linear of every layer; for the prefill a few rows for
every token, and a row of every 32-row quadrant of every 128-row tile for sixteen tokens."""
import numpy as np
import pytest
import torch

import oracle
from paper_2602_04163_b200 import binding, synth
from tests import gpu_util as G

pytestmark = pytest.mark.gpu

SHAPES = synth.QWEN25_72B_LAYER
GROUP = 128


def _sample_rows(out: int, salt: int, n: int = 3) -> np.ndarray:
    """First and last row plus n rows that move with `salt` (plain arithmetic, no generator state)."""
    moving = [(salt * 7919 + k * 104729 + 13) % out for k in range(n)]
    return np.unique(np.array([0, out - 1] + moving, dtype=np.int64))


def test_decode_sweep_80_layers():
    K, n_layers, base_seed = 2, 80, 5
    sp = G.stream_ptr()
    hs = [[binding.Handle(o, i, K, GROUP, None, synth.linear_seed(base_seed, layer, li, K), 1)
           for li, (_, o, i) in enumerate(SHAPES)] for layer in range(n_layers)]
    assert sum(h.packed_bytes for L in hs for h in L) == n_layers * 260_554_752
    xb = {i: synth.activations(9, 1, i) for i in (8192, 29568)}
    xs = {i: G.x_tensor(v) for i, v in xb.items()}
    y_single = [[torch.full((1, o), float("nan"), dtype=torch.float16, device="cuda") for _, o, _ in SHAPES] for _ in range(n_layers)]
    y_batch = [[torch.full((1, o), float("nan"), dtype=torch.float16, device="cuda") for _, o, _ in SHAPES] for _ in range(n_layers)]
    for layer in range(n_layers):                                   # the benchmark's first form: 560 calls, nothing waits in between
        for li, h in enumerate(hs[layer]):
            h.bpdq_linear(xs[h.in_].data_ptr(), y_single[layer][li].data_ptr(), 1, sp)
    for layer in range(n_layers):                                   # its second form: one launch per layer
        binding.bpdq_linear_batch(hs[layer], [xs[h.in_].data_ptr() for h in hs[layer]],
                                  [y.data_ptr() for y in y_batch[layer]], 1, sp)
    torch.cuda.synchronize()
    worst = 0.0
    for layer in range(n_layers):
        for li, (name, o, i) in enumerate(SHAPES):
            hs[layer][li].bpdq_get_status(sp)
            seed = synth.linear_seed(base_seed, layer, li, K)
            rows = _sample_rows(o, layer * 7 + li)
            y_ref, a_ref = oracle.linear(synth.plane_bits(seed, o, i, K, rows), synth.coefficients(seed, o, i, K, GROUP, rows), xb[i], GROUP)
            for what, ys in (("single", y_single), ("batch", y_batch)):
                y = ys[layer][li].cpu().numpy().astype(np.float64)
                assert np.all(np.isfinite(y)), f"layer {layer} {name} {what}"
                worst = max(worst, G.assert_linear_close(y[:, rows], y_ref, a_ref, f"layer {layer} {name} {what}"))
    # two linears through the device blob itself: read it back, decode it with the checker's own reader
    for layer, li in ((37, 1), (79, 3)):
        name, o, i = SHAPES[li]
        bits, coef = oracle.unpack(hs[layer][li].bpdq_read_blob(), o, i, K, GROUP)
        rows = _sample_rows(o, 1000 + layer, n=6)
        y_ref, a_ref = oracle.linear(bits[:, rows], coef[:, rows], xb[i], GROUP)
        y = y_batch[layer][li].cpu().numpy().astype(np.float64)
        G.assert_linear_close(y[:, rows], y_ref, a_ref, f"layer {layer} {name} from the blob")
        del bits, coef
    assert worst < 1.0
    for L in hs:
        for h in L:
            h.bpdq_destroy()


def _tile_quadrant_rows(out: int) -> np.ndarray:
    """One row in every 32-row quadrant of every 128-row tile, its position inside the quadrant moving with the tile."""
    rows = []
    for tile in range((out + 127) // 128):
        for quad in range(4):
            r = tile * 128 + quad * 32 + (tile * 5 + quad * 11) % 32
            if r < out:
                rows.append(r)
    return np.unique(np.array(rows + [0, out - 1], dtype=np.int64))


@pytest.mark.parametrize("K,M", [(3, 8192)])
def test_prefill_layer(K, M):
    sp = G.stream_ptr()
    tok16 = np.unique(np.array([0, 255, 256, M - 1] + [(k * 2654435761 + 977) % M for k in range(12)], dtype=np.int64))
    xbs, xds = {}, {}
    for i in sorted({i for _, _, i in SHAPES}):                     # the benchmark's activations: one tensor per input width
        xbs[i] = np.concatenate([synth.activations(3, M, i, tokens=np.arange(t0, min(M, t0 + 512))) for t0 in range(0, M, 512)])
        xds[i] = G.x_tensor(xbs[i])
    for li, (name, o, i) in enumerate(SHAPES):
        seed = 700 + li                                             # the benchmark's handles
        h = binding.Handle(o, i, K, GROUP, None, seed, M)
        xb, x = xbs[i], xds[i]
        y = torch.full((M, o), float("nan"), dtype=torch.float16, device="cuda")
        h.bpdq_linear(x.data_ptr(), y.data_ptr(), M, sp)            # the dispatcher's choice, as in the benchmark
        torch.cuda.synchronize()
        h.bpdq_get_status(sp)
        assert bool(torch.isfinite(y).all()), name
        # every token, a few rows
        rows = _sample_rows(o, li, n=0 if i > 8192 else 1)
        y_ref, a_ref = oracle.linear(synth.plane_bits(seed, o, i, K, rows), synth.coefficients(seed, o, i, K, GROUP, rows), xb, GROUP)
        G.assert_linear_close(y[:, torch.from_numpy(rows).cuda()].cpu().numpy().astype(np.float64), y_ref, a_ref, f"{name} all tokens")
        # every tile and quadrant, sixteen tokens
        rows = _tile_quadrant_rows(o)
        y_ref, a_ref = oracle.linear(synth.plane_bits(seed, o, i, K, rows), synth.coefficients(seed, o, i, K, GROUP, rows), xb[tok16], GROUP)
        got = y[torch.from_numpy(tok16).cuda()][:, torch.from_numpy(rows).cuda()].cpu().numpy().astype(np.float64)
        G.assert_linear_close(got, y_ref, a_ref, f"{name} all tiles")
        h.bpdq_destroy()
        del y
