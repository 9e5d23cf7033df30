"""B200-native fused linear layers (libmtmcfused): Y = epilogue(X.W^T + b).

The Python side is argument marshalling only; every step of the path runs in the
hand-written sm_100a kernels behind the C-ABI library (see include/mtmc_fused.h).
Importing this package does not load the library; the first call does, and it
raises if the library or a Blackwell GPU is missing -- there is no fallback.
"""
__all__ = ["inputs"]
