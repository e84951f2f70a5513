"""B200-native {-1,+1} bit-plane quantized layers: encode, branch-fused binary GEMM, conv.

The CUDA library (``libmpq.so``, built from ``csrc/``) is loaded on first use by
:mod:`paper_1905_13389_b200.binding`; there is no CPU fallback.
"""
