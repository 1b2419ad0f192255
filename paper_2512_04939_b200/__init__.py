"""B200-native geometry-aware cached token merging around VGGT's global attention.

The package is a thin ctypes binding over ``liblitevggt.so`` (hand-written sm_100a CUDA
kernels behind a C ABI, declared in ``include/litevggt.h``).  There is no CPU or
pure-PyTorch fallback: importing :mod:`paper_2512_04939_b200.binding` fails loudly when
the library has not been built (``python -m paper_2512_04939_b200.build``).
"""
from .binding import (  # noqa: F401
    LiteVGGT,
    LiteVGGTError,
    Plan,
    CLS_PROTECTED,
    CLS_GA,
    CLS_DST,
    CLS_SRC,
    global_attn_static,
    STATIC_ATTN_MAX_ROWS,
    library_path,
    load_library,
)
