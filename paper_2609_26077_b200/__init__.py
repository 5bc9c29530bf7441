"""B200-native block-scaled e4m3 fast matrix multiplication (rank-7 2x2 realizations).

The compute lives in libfmm_b200.so (hand-written CUDA for sm_100a behind the C ABI of
include/fmm.h); `fmm` is the ctypes binding, `realizations` the coefficient tables and
`workloads` the seeded synthetic operand generators.  Nothing is loaded at import time.
"""
__all__ = ["fmm", "realizations", "workloads", "build"]
