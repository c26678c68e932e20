"""B200-native k-MIP self-attention (hot path): thin Python binding over a C-ABI CUDA library."""
