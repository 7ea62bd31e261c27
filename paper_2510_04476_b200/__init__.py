"""B200-native CCA / CCGQA attention block: C-ABI CUDA library plus a thin ctypes binding."""
