"""Group-wise int8-quantized Winograd convolution F(m,3) for NVIDIA B200 (sm_100a).

``workloads``  seeded synthetic layers (no method arithmetic)
``binding``    thin ctypes binding of the C-ABI library ``libwfq.so`` (CUDA kernels)
``build``      nvcc build of the library

The package never falls back to a CPU implementation: ``binding`` raises if the
CUDA library is missing.
"""
__all__ = ["workloads", "binding", "build"]
