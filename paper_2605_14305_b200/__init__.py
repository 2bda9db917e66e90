"""B200-native speculative verification for FeF-DLLM decoding (binding added with the CUDA library)."""
