"""B200-native 8-bit quantized CNN inference primitives (C ABI in include/q8.h, kernels in csrc/)."""
from .binding import *  # noqa: F401,F403
from .binding import lib, EXPORTS, Q8Error, q8_conv_desc  # noqa: F401
