"""B200-native NVFP4 quantize-then-GEMM hot path (C-ABI CUDA library + thin binding)."""
