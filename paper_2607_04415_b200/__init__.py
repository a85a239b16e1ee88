"""GPU-owned paged graph beam search for B200 (sm_100a).

Thin Python binding over the C ABI in include/gorio.h.  Every step of the search runs in
the CUDA kernels of libgorio.so; this package only marshals arguments.  There is no CPU
fallback: calls raise if the library has not been built (python -m paper_2607_04415_b200.build).
"""
from .binding import (  # noqa: F401
    GorioError,
    Index,
    Stats,
    lib_path,
    load_library,
    EXPORTED_SYMBOLS,
    search_resident_noalloc,
)
