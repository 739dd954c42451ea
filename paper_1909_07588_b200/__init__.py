"""B200-native LAQ (lazily aggregated quantized gradients) hot path: CUDA library + thin binding."""
