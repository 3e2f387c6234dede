"""B200-native 2:4 structured-sparse GEMM path (arXiv 2104.08378): prune, compress, sparse GEMM.

The package is a thin binding over the C-ABI library built from ``csrc/`` (see ``include/sp24.h``).
``inputs`` (numpy-only synthetic workloads) can be imported without the CUDA library; everything
in ``binding`` loads ``libsp24.so`` and fails loudly if it is missing.
"""
__all__ = ["inputs", "binding"]
