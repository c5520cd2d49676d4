"""B200-native SPECTRE spectral-mixer library (C-ABI CUDA kernels + thin binding)."""
