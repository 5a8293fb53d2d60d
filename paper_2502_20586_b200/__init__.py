"""B200-native MXFP4 linear-layer backward: blockwise RHT + SR quantiser and block-scaled FP4 GEMM.

``paper_2502_20586_b200.binding`` is the thin Python view of the C-ABI library
(``include/mxfp4.h``); ``paper_2502_20586_b200.workloads`` holds shapes and seeded input
generators.  Importing the package does not load the CUDA library; importing
``binding`` does, and raises if it has not been built.
"""
