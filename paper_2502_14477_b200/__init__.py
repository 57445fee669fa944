"""B200 (sm_100a) library for one step of Efficient Selective Attention.

The arithmetic lives in the CUDA library ``libesa_b200.so`` (C ABI declared in
``include/esa.h``); this package only marshals arguments.  There is no CPU or
PyTorch fallback: without the built library every call raises.
"""
from .binding import (  # noqa: F401
    EsaError,
    EsaConfig,
    Esa,
    EsaFit,
    load_library,
    library_path,
    STATUS_NAMES,
    attend_noalloc,
)
from .build import build_library  # noqa: F401

__all__ = ["EsaError", "EsaConfig", "Esa", "EsaFit", "load_library", "library_path", "build_library", "STATUS_NAMES", "attend_noalloc"]
