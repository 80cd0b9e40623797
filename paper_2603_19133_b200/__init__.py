"""B200-native hot path of PicoSpec's separate rejection sampling with sparse compression:
a C-ABI CUDA library (csrc/, include/picospec.h) and this thin ctypes binding."""
from .binding import (BF16, CHUNK, EDATA, F32, OK, STATIC_MAX_ROWS, STATIC_MAX_VOCAB, Context, PicospecError,
                      lib, verify_static, wire_bytes)  # noqa: F401
from . import perf_model  # noqa: F401
from .buildlib import build  # noqa: F401
