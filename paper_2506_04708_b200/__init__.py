"""STAND speculative-sampling hot path for B200 (sm_100a).

`inputs` holds the seeded synthetic workloads.  `binding` holds the thin ctypes
layer over the C-ABI library (`include/stand.h`); it loads the CUDA library on
first use and raises if the library has not been built.
"""
