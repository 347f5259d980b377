"""B200-native quantized-and-cached DiT denoising step (Q&C, arXiv 2503.02508).

The work is done by libqdit.so (hand-written sm_100a CUDA behind a C ABI, see
include/qdit.h).  This package is only the ctypes binding: it marshals torch
tensors (used for device memory and streams) into pointers.  Importing it
without the built library raises ImportError; there is no fallback path.
"""
from .binding import *  # noqa: F401,F403
from .binding import __all__  # noqa: F401
