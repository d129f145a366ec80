"""Runs one kernel of the library a few times on one synthetic layer (for use under a profiler).

    python -m paper_2602_04163_b200.profile_case --kernel gemv --out 59136 --in 8192 --K 2 --M 1 --iters 3

--kernel is one of gemv, gemm, simple, auto, dequant, or layer72b (the seven linears of a
Qwen2.5-72B-shaped decoder layer in one bpdq_linear_batch launch; --out/--in are ignored).  Weights are generated on the device from
--seed; activations come from the seeded host generator.  Prints the median time of the timed
launches (CUDA events) so that the same command is also a quick stand-alone measurement.
"""
from __future__ import annotations

import argparse

import numpy as np
import torch

from . import binding, synth

KERNELS = {"auto": binding.KERNEL_AUTO, "gemv": binding.KERNEL_GEMV, "gemm": binding.KERNEL_GEMM,
           "simple": binding.KERNEL_GEMV_SIMPLE}


def main() -> None:
    ap = argparse.ArgumentParser()
    ap.add_argument("--kernel", default="gemv", choices=sorted(KERNELS) + ["dequant", "layer72b"])
    ap.add_argument("--out", type=int, default=29568)
    ap.add_argument("--in", dest="in_", type=int, default=8192)
    ap.add_argument("--K", type=int, default=2)
    ap.add_argument("--group", type=int, default=128)
    ap.add_argument("--M", type=int, default=1)
    ap.add_argument("--iters", type=int, default=3)
    ap.add_argument("--seed", type=int, default=1)
    ap.add_argument("--flush-l2", action="store_true", help="write 256 MB between launches")
    a = ap.parse_args()

    torch.cuda.set_device(0)
    stream = torch.cuda.current_stream()
    sp = stream.cuda_stream
    if a.kernel == "layer72b":
        run_layer(a, stream)
        return
    h = binding.Handle(a.out, a.in_, a.K, a.group, None, a.seed, max(1, a.M))
    x = torch.from_numpy(synth.activations(a.seed + 1, a.M, a.in_).view(np.int16).copy()).cuda().view(torch.float16)
    y = torch.empty((a.M, a.out), dtype=torch.float16, device="cuda")
    w = torch.empty((a.out, a.in_), dtype=torch.float16, device="cuda") if a.kernel == "dequant" else None
    flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda") if a.flush_l2 else None

    def call():
        if a.kernel == "dequant":
            h.bpdq_dequant(w.data_ptr(), sp)
        else:
            h.bpdq_linear_ex(x.data_ptr(), y.data_ptr(), a.M, KERNELS[a.kernel], sp)

    times = []
    for _ in range(a.iters):
        if flush is not None:
            flush.zero_()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        call()
        e1.record(stream)
        e1.synchronize()
        times.append(e0.elapsed_time(e1))
    h.bpdq_get_status(sp)
    times.sort()
    med = times[len(times) // 2]
    packed = h.packed_bytes
    flops = 2.0 * a.M * a.in_ * a.out
    print(f"{a.kernel} out={a.out} in={a.in_} K={a.K} g={a.group} M={a.M}: median {med * 1e3:.1f} us over {a.iters} "
          f"launches; packed {packed / 1e6:.1f} MB -> {packed / med / 1e6:.0f} GB/s; {flops / med / 1e9:.1f} TFLOP/s")
    h.bpdq_destroy()


def run_layer(a, stream) -> None:
    sp = stream.cuda_stream
    shapes = synth.QWEN25_72B_LAYER
    hs = [binding.Handle(o, i, a.K, a.group, None, a.seed + li, max(1, a.M)) for li, (_, o, i) in enumerate(shapes)]
    xs = {i: torch.from_numpy(synth.activations(a.seed + 9, a.M, i).view(np.int16).copy()).cuda().view(torch.float16)
          for i in sorted({i for _, _, i in shapes})}
    ys = [torch.empty((a.M, o), dtype=torch.float16, device="cuda") for _, o, _ in shapes]
    flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda") if a.flush_l2 else None
    times = []
    for _ in range(a.iters):
        if flush is not None:
            flush.zero_()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        binding.bpdq_linear_batch(hs, [xs[h.in_].data_ptr() for h in hs], [y.data_ptr() for y in ys], a.M, sp)
        e1.record(stream)
        e1.synchronize()
        times.append(e0.elapsed_time(e1))
    times.sort()
    med = times[len(times) // 2]
    packed = sum(h.packed_bytes for h in hs)
    print(f"layer72b batch K={a.K} g={a.group} M={a.M}: median {med * 1e3:.1f} us over {a.iters} launches; "
          f"packed {packed / 1e6:.1f} MB -> {packed / med / 1e6:.0f} GB/s")
    for h in hs:
        h.bpdq_destroy()


if __name__ == "__main__":
    main()
