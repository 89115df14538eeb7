"""B200-native forward pass of one Tucker-factorised attention layer (prefill + cached decode).

The compute lives in a C-ABI CUDA library (csrc/, declared in include/tucker_attn.h); the
Python side only marshals arguments.  Importing this package loads nothing native; the
library is loaded on first use and a missing build raises instead of falling back.
"""
__all__ = ["workloads"]
