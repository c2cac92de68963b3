"""Single-GPU Parle round (arXiv 1707.00424, Section 3) on hand-written sm_100a
kernels behind a C ABI (include/parle.h).  This package is the thin ctypes
binding; every step of the round runs in the CUDA library."""
from .binding import (  # noqa: F401
    GEMM_BF16, GEMM_FP32, FLAG_BAD_LABEL, FLAG_NONFINITE, FLAG_WAIT_LIMIT,
    ParleError, Parle, lib, library_path, softmax_ce_static, STATIC_LOSS_MAX_ROWS, scoping,
)
