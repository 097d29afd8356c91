"""B200-native fused low-bit (SOLO) optimizer step: C-ABI CUDA library + thin binding."""
