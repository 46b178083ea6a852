"""B200-native WeightedKV decode hot path: C-ABI CUDA library plus a thin ctypes binding."""
