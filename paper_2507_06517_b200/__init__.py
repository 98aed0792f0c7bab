"""B200-native SpindleKV prefill KV-cache reduction pass (CUDA library + thin binding)."""
