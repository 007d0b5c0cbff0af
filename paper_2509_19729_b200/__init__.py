"""B200-native TP a->b re-layout of an LLM instance's state (paged KV cache + projection weights).

The work is done by hand-written sm_100a CUDA kernels behind a C ABI (``include/amoeba.h``); this package is the
thin ctypes binding with the same function names.  There is no CPU fallback: if the shared library cannot be
loaded the import fails.
"""
from .binding import *  # noqa: F401,F403
from .binding import __all__  # noqa: F401
