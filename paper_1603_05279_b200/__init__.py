"""B200-native forward path of the XNOR-Net binary convolution block.

The work is done by libxnor.so (hand-written CUDA for sm_100a behind a C ABI,
declared in include/xnor.h); this package is its ctypes binding plus the shape
tables and seeded input generators of the benchmark workloads.
"""
from . import workloads  # noqa: F401
from .binding import *  # noqa: F401,F403
from .binding import load, make_desc, desc_of, XnorError, xnor_conv_desc  # noqa: F401
