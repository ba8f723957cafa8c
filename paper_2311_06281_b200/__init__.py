"""B200-native fused evaluation of x_t = a_t*x_{t-1} + b_t through the two-prefix-sum
log-space expression of Heinsen (2023), Eq. 1-3 and Eq. 7-8.

The product is the C-ABI library ``libheinsen_scan.so`` (hand-written sm_100a CUDA
kernels, sources under ``csrc/``, declarations in ``include/heinsen_scan.h``).
``heinsen_scan`` is the thin Python binding over it; ``workloads`` draws the seeded
synthetic inputs.  Importing the package does not load the library; the first call
does, and fails loudly if it has not been built.
"""
__all__ = ["heinsen_scan", "workloads", "build_ext", "sharding"]
