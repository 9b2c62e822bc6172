"""B200-native selective-recompute prefill with probe-guided per-unit KV offset correction.

The package is a thin binding over `libakvs.so` (hand-written sm_100a CUDA kernels behind a
C ABI, declared in include/akvs.h).  Importing it loads the library and fails loudly when
the library has not been built; there is no fallback implementation.
"""
from . import binding
from .binding import *  # noqa: F401,F403
