"""bpdq_linear_noalloc, the entry point for callers that cannot allocate device memory.

Collected last on purpose: a run that stops at the first failure has then already run every other
test.  The entry point works on a caller-owned device blob with the library's static scratch; its
output must agree with the handle-based look-up-table kernel on the same weights, on two calls in
a row (the second call finds the scratch as the first one left it).
"""
import numpy as np
import pytest

from paper_2602_04163_b200 import binding, synth
from tests import gpu_util as G

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("K,g,out,in_,M", [(2, 128, 4096, 4096, 1), (3, 128, 272, 896, 3), (2, 256, 64, 1024, 2),
                                            (1, 128, 65536, 128, 3)])     # the most rows it takes: last counter, last scratch row, two passes
def test_noalloc_matches_handle_kernel_twice(K, g, out, in_, M):
    import torch
    h, bits, coef = G.make_layer(80 + K, out, in_, K, g, max_M=M)
    xb = synth.activations(81, M, in_)
    y_ref = G.run_linear(h, xb, binding.KERNEL_GEMV)                  # existing entry point, handle-owned scratch
    blob = torch.from_numpy(binding.bpdq_pack(bits, coef, g)).cuda()   # caller-owned device copy of the packed weights
    x = G.x_tensor(xb)
    for call in range(2):
        y = torch.full((M, out), float("nan"), dtype=torch.float16, device="cuda")
        binding.bpdq_linear_noalloc(blob.data_ptr(), out, in_, K, g, x.data_ptr(), y.data_ptr(), M, G.stream_ptr())
        torch.cuda.synchronize()
        got = y.cpu().numpy().astype(np.float64)
        # the two kernels add the same binary32 partial sums in a free order: last binary16 digit at most
        assert np.allclose(got, y_ref, rtol=2.0 ** -9, atol=1e-5), f"call {call}"
    # and against the checker, with the bound every linear kernel is held to
    import oracle
    yo, ao = oracle.linear(bits, coef, xb, g)
    G.assert_linear_close(got, yo, ao, "noalloc")


def test_noalloc_rejects_what_it_cannot_hold():
    import torch
    x = torch.zeros(256, dtype=torch.float16, device="cuda")
    big = binding.NOALLOC_MAX_OUT + 16
    with pytest.raises(binding.BpdqError) as ei:
        binding.bpdq_linear_noalloc(x.data_ptr(), big, 128, 2, 128, x.data_ptr(), x.data_ptr(), 1, G.stream_ptr())
    assert ei.value.code == binding.ERR_INVALID and "static scratch" in str(ei.value)
    with pytest.raises(binding.BpdqError) as ei:
        binding.bpdq_linear_noalloc(x.data_ptr(), 64, 128, 2, 128, x.data_ptr(), x.data_ptr(), binding.GEMV_MAX_M + 1, G.stream_ptr())
    assert ei.value.code == binding.ERR_INVALID
    binding.bpdq_linear_noalloc(0, 64, 128, 2, 128, 0, 0, 0, G.stream_ptr())      # M = 0: nothing to do
