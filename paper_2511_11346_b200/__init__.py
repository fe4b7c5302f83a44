"""B200 (sm_100a) implementation of the MtPC probabilistic-circuit multi-byte prediction head.

`binding` is the ctypes layer over the C ABI in include/mtpc.h; `inputs` draws the seeded synthetic workloads.
The CUDA library is loaded on first use and there is no fallback path.
"""
