"""Generalized PolyDot coded matrix multiplication on B200 (sm_100a): Python face of libgpd.so.

The names mirror the C ABI declared in include/gpd.h.  Importing the package loads the CUDA
library; it fails loudly when the library has not been built (there is no CPU fallback).
"""

from .binding import *  # noqa: F401,F403
from .binding import EXPORTED, Plan, GpdError, lib, new_results, read_results, result_slot  # noqa: F401
