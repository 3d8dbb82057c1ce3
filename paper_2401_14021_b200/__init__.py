"""B200-native exact dense retrieval for RaLMSpec-style serving (CUDA, sm_100a).

Thin ctypes binding over the C ABI in include/ralm.h. Every step runs in the CUDA
library; torch is used for device memory and streams only. There is no CPU fallback: if
the compiled library is missing or no CUDA device is present, calls raise.
"""
from .binding import (IP, L2, Index, RalmError, cache_search, cache_update, merge_lists, lib_path, load_library, search,
                      search_host, search_static, verify, os3_gamma, os3_stride, STATUS_NAMES)

__all__ = ["IP", "L2", "Index", "RalmError", "cache_search", "cache_update", "merge_lists", "lib_path", "load_library", "search",
           "search_host", "search_static", "verify", "os3_gamma", "os3_stride", "STATUS_NAMES"]
