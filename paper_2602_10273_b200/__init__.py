"""B200-native Power-SMC step: CUDA kernels behind a C-ABI, with a thin ctypes binding."""
