"""B200 (sm_100a) implementation of one AdaCGD iteration behind a C ABI.

The Python layer only marshals arguments: every step of the path runs in the CUDA
kernels of libadacgd.so.  Importing this package does not need a GPU; calling it does,
and there is no CPU fallback.
"""
from .binding import (  # noqa: F401
    AdaCGD, Cand, TOPK, QUANT, LOSS_LOGISTIC_NCVX, LOSS_LOGISTIC_L2, LOSS_LEAST_SQUARES, LOSS_NONE,
    AdacgdError, load_library, EXPORTED_SYMBOLS, compress_noalloc, NOALLOC_MAX_ROWS, NOALLOC_MAX_D, message_bits,
    PRED_LAZY, PRED_ABSOLUTE, PRED_RELATIVE, PRED_NEVER, PRED_ALWAYS,
)
from . import protocol  # noqa: F401,E402
