"""B200-native chunkwise hard-routing prefill of SMat-Attention (C-ABI CUDA library + thin binding)."""
