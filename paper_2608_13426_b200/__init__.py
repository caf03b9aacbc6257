"""B200-native (sm_100a) hot path of Reduced Matrix Multiplication (RMM).

The product is the C-ABI library librmm_b200.so (include/rmm.h); this package is its thin ctypes
binding plus the seeded input generators (synth).  Importing the package does not need a GPU; calling
any rmm_* function does, and raises if the shared library has not been built.
"""
from . import synth  # noqa: F401
from .binding import (  # noqa: F401
    RmmError,
    rmm,
    rmm_debug_control,
    rmm_keep_count,
    rmm_launch_count,
    rmm_product,
    rmm_product_host,
    rmm_reduced_attn,
    rmm_reduced_gemm,
    rmm_reduced_gemm_q8,
    rmm_score,
    rmm_score_select,
    rmm_score_select_static,
    rmm_score_select_static_capacity,
    rmm_score_select_static_status,
    rmm_select,
    rmm_status_read,
)
