"""Filtered convolution backward pass of gradient filtering on B200 (sm_100a).

A thin binding over the C ABI of libgf_b200.so (include/gf.h).  The CUDA
library is the only implementation: nothing here computes on the CPU.
"""
from . import workloads  # noqa: F401
from .binding import *  # noqa: F401,F403
from .binding import build_library, lib, library_path  # noqa: F401
from .autograd import FilteredConv2d, filtered_conv2d  # noqa: F401
