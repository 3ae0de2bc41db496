"""B200-native delta attention (DeltaLLM hot path): CUDA library + thin Python binding."""
