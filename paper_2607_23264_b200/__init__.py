"""B200-native (sm_100a) MoE forward at EP=1: routing plan, dispatch, SwiGLU expert grouped GEMM, combine.

Importing the package does not load the CUDA library; ``paper_2607_23264_b200.binding`` does, and
fails loudly when it has not been built (there is no CPU fallback).
"""
