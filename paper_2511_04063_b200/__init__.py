"""B200-native rotational distribution calibration (DartQuant's calibration step).

The product is libdartquant.so (hand-written sm_100a CUDA behind a C ABI, see
include/dartquant.h); this package is its thin Python binding plus the seeded
synthetic-input generators.  Importing the package does not load the library;
calling any dq_* function does, and raises if it is not built.
"""
from . import inputs  # noqa: F401
from .binding import *  # noqa: F401,F403
from .binding import (DartQuantError, EXPORTED_SYMBOLS, LIB_PATH, dq_calib_config,  # noqa: F401
                      load_library, status_string)
