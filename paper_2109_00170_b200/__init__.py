"""SIMD-structured sparse pointwise convolution on NVIDIA B200: Python binding of the C-ABI
library (libalcs.so, built from csrc/ for sm_100a).  The binding only marshals arguments."""
from .binding import *  # noqa: F401,F403
from .binding import lib, LIB_PATH, EXPORTS, AlcsError, LaunchCfg, Packed, Stack  # noqa: F401
