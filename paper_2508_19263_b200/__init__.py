"""B200-native lossless exponent / sign+mantissa Huffman codec for BF16, FP8 (E4M3, E5M2) and FP4 E2M1 tensors.

``binding``   ctypes access to the C ABI of ``libzc.so`` (CUDA kernels + host logic)
``build``     compiles ``libzc.so`` in-tree with nvcc for sm_100a
``workloads`` seeded synthetic input tensors (no codec arithmetic)
"""
__all__ = ["binding", "build", "workloads"]
