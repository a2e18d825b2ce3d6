"""B200-native GEMM + all-scatter over an emulated symmetric heap (arXiv 2511.12500's hot path).

The product is the C-ABI library (include/iris_b200.h); this package is its thin ctypes binding.
"""
from .binding import *  # noqa: F401,F403
from .binding import EXPORTS, LIB_PATH, IrisError, lib  # noqa: F401
