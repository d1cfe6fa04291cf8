"""B200-native FPROP direct convolution (maxDNN's hot path) — Python binding.

The product is the C-ABI library ``libmaxdnn.so`` (declared in
``include/maxdnn.h``); this package only marshals arguments to it.  Importing
the package is cheap; the library is loaded on first use and a missing library
raises — there is no CPU fallback.
"""
from . import workloads  # noqa: F401
from .binding import *  # noqa: F401,F403
from .binding import __all__ as _binding_all

__all__ = ["workloads"] + list(_binding_all)
