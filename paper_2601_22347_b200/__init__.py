"""PeRQ online path (permute, block-Hadamard rotate, quantise to INT4 / MXFP4) for NVIDIA B200.

The product is the CUDA library `libperq.so` (C ABI in include/perq.h); `binding` exposes
the same entry points to Python.  `inputs` holds the seeded synthetic workloads and
`roofline` the byte/op model used to report bandwidth.
"""
