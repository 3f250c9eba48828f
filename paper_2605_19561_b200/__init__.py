"""B200-native hot path of TORQ's rotated-MXFP4 linear layer (rotate -> MXFP4 quantize
-> block-scaled FP4 GEMM) behind a C-ABI shared library; this package is the thin
Python binding plus the seeded input generators."""
