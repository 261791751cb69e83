"""B200-native DoubleSqueeze step: ctypes binding over the C-ABI CUDA library."""
from .binding import DoubleSqueeze, DsqError, load_library  # noqa: F401
from .workloads import Q, WORKLOADS, Workload, make_gradients  # noqa: F401
