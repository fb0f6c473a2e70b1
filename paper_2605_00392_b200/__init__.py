"""B200-native RTPrune visual-token pruning: CUDA kernels behind a C ABI, with a thin binding."""
