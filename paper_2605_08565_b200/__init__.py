"""B200-native block-scaled FP4 quantization, scale search and MSE scoring (libmxq).

``binding``  ctypes binding of the C-ABI in ``include/mxq.h`` (CUDA only, no fallback)
``inputs``   seeded synthetic input generators (no quantization arithmetic)
``build``    in-tree nvcc build of ``libmxq.so``
"""
__all__ = ["binding", "inputs", "build"]
