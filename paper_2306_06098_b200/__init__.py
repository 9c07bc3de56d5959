"""B200-native EFCP / Sparse M-FAC hot path: Python binding over the C-ABI CUDA library."""
