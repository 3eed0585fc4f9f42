"""CDL quantized layer on B200: Python face of the C-ABI library ``libcdl.so``.

The functions re-exported here marshal arguments only; every step of the path
runs in the CUDA kernels of ``csrc/``.  The library is loaded on first use and
a missing build raises: there is no CPU or PyTorch fallback.
"""
from .api import *  # noqa: F401,F403
from .api import __all__  # noqa: F401
