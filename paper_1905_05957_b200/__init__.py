"""B200-native DoubleSqueeze step: ctypes binding over the C-ABI CUDA library."""
