"""Tree-verification step of speculative decoding for one B200 GPU.

The work is done by hand-written CUDA kernels behind the C-ABI declared in
``include/ghd.h`` (built into ``libghd.so`` next to this file).  This package is
the thin Python binding: it marshals torch tensors into that ABI and nothing
else - there is no CPU or PyTorch fallback, and importing the binding fails
loudly when the library is missing.
"""
from .binding import *  # noqa: F401,F403
from .binding import __all__  # noqa: F401
