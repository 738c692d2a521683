"""B200-native SAMA meta-gradient step (arXiv 2310.05674): C-ABI CUDA library plus a thin binding."""
