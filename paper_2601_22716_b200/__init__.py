"""B200-native LoRDS dequantize-and-multiply: y = x (L[Q] (.) (B A))^T behind a C ABI.

``binding`` holds the Python names of the C entry points (include/lords.h); ``inputs``
draws the seeded synthetic layers; ``packing`` lays several layers over one input out as
one layer; ``build`` compiles the CUDA library in-tree.
Nothing here computes on the CPU: the hot path exists only as sm_100a kernels.
"""
__all__ = ["binding", "inputs", "packing", "build"]
