"""B200-native TABED speculative-decoding round: a C library of sm_100a CUDA kernels
(csrc/, include/tabed.h) and a thin ctypes binding (binding.py).  workloads.py draws the seeded
synthetic inputs; it contains none of the method's arithmetic."""
