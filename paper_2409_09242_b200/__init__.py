"""B200-native batched AdaHessian + elastic-averaging round (arXiv 2409.09242).

``binding`` is the thin ctypes layer over the C-ABI CUDA library (include/adahess.h);
``workloads`` holds the synthetic layouts and seeded input buffers.  There is no CPU
fallback: importing ``binding`` without the built library raises.
"""
__all__ = ["binding", "workloads", "build"]
