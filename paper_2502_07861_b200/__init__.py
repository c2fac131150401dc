"""BalanceKV hot path on B200: C-ABI CUDA library plus a thin ctypes binding."""
