"""SCAP sparse fully-connected layer for NVIDIA B200 (sm_100a).

The product is the C-ABI library ``libscap_b200.so`` (declared in ``include/scap.h``); this package
is its thin Python binding: the functions below have the names and argument order of the C entry
points, take torch CUDA tensors (or CPU tensors for the host-buffer call), and do argument
marshalling only.  There is no CPU or PyTorch fallback: if the library has not been built, the
first call raises.
"""
from .binding import *  # noqa: F401,F403
from .binding import __all__  # noqa: F401
