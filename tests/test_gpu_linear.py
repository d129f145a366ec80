"""bpdq_linear (all kernels) against the checker: |y - y_ref| <= 4e-3 * sum|x w| + 1e-3 per element."""
import numpy as np
import pytest

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
