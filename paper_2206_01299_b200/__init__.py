"""AQ-SGD activation-delta codec for one B200: CUDA library + thin ctypes binding."""
from .binding import *  # noqa: F401,F403
from .binding import lib, AqError, SIGNATURES, LIB_PATH  # noqa: F401
