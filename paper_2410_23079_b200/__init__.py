"""libbuzz: the BUZZ sparse KV-cache hot path (prefill scoring, decode attention, eviction) as
hand-written CUDA for sm_100a behind a C ABI, with a thin ctypes binding."""
from .binding import (BUZZ_BF16, BUZZ_F32, BUZZ_FLAG_LOGN, Buzz, BuzzError, error_string,  # noqa: F401
                      exported_symbols, load_library)
