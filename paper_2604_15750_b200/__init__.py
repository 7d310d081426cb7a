"""DepCap block-step on B200: Python binding over the C-ABI CUDA library (libdepcap.so).

Argument marshalling only; every step of the path runs in the library's kernels.
"""
from .binding import (DepCap, DepCapError, Hyper, lib, load_library, pack_kv_cache,  # noqa: F401
                      STAGE_NAMES, signals_static)
