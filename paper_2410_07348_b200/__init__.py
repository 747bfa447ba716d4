"""MoE++ heterogeneous expert layer, forward pass, for NVIDIA B200 (sm_100a).

The product is the C-ABI library declared in ``include/moepp.h`` (built from ``csrc/``); this package
is its thin Python binding plus the seeded workload generators.  Importing the package is cheap and
loads nothing; the shared library is loaded on first use and a missing library is a hard error.
"""
__all__ = ["workloads"]
