"""B200 (sm_100a) implicit-ALS half-epoch library: CUDA kernels behind a C ABI, plus a thin binding."""
from .binding import (ALX_BF16, ALX_COLS, ALX_DEFAULT_SPLIT, ALX_F32, ALX_N_CLASSES, ALX_ROWS, Alx, AlxError,
                      load_library)

__all__ = ["Alx", "AlxError", "load_library", "ALX_ROWS", "ALX_COLS", "ALX_F32", "ALX_BF16", "ALX_N_CLASSES",
           "ALX_DEFAULT_SPLIT"]
