"""B200 (sm_100a) library for the leapfrog backward pass of a sigmoid MLP (arXiv 1801.04928).

The work is done by hand-written CUDA kernels behind the C ABI of ``include/leapfrog.h``;
this package is the ctypes binding.  Importing it requires the built ``libleapfrog.so``.
"""
from .binding import *  # noqa: F401,F403
from .binding import Leapfrog, LeapfrogError, EXPORTS, LIB_PATH  # noqa: F401
