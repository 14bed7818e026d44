"""B200-native Lag-Relative Sparse Attention (LRSA) hot path: CUDA kernels behind a C ABI.

``paper_2506_11498_b200.lrsa`` is the thin binding over the shared library;
``paper_2506_11498_b200.workloads`` holds the seeded synthetic inputs.
Nothing is loaded at import time.
"""
