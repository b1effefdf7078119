"""B200-native Strassen-Winograd (CAPS single-GPU hot path)."""
