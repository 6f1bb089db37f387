"""B200-native hot path of AET-SGD (arXiv 2112.13935): clients' local-SGD
rounds under s_i = a*i + b and the server's delay-aware ordered aggregation,
as a C-ABI CUDA library (include/aet.h) with a thin ctypes binding."""
from . import workloads  # noqa: F401
