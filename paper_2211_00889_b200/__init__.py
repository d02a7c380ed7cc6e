"""B200-native Non-blocking SGD aggregate-and-update path (C-ABI library + thin ctypes binding)."""
