"""B200-native Batch Normalization Sampling (arXiv 1810.10962): thin Python binding over the C-ABI
CUDA library ``libbns.so``.  Import ``paper_1810_10962_b200.bns`` for the calls; this package does
no arithmetic of its own and has no CPU fallback."""
