"""B200-native FP8 hot path (E4M3 / E5M2 casts and FP8 GEMMs) behind a C ABI."""
