"""BPDQ weight-only linear layer for NVIDIA B200: CUDA kernels behind a C ABI (libbpdq.so).

`binding` is the thin ctypes layer over include/bpdq.h; `synth` draws seeded synthetic inputs;
`build` compiles the library in-tree.  Nothing here computes on the CPU.
"""
