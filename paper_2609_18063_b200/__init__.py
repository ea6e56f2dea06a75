"""B200-native streaming-MoE per-layer decode step: thin ctypes binding over the CUDA library.

Importing this package loads ``libedgmoe.so`` (built in-tree by ``build.build()``); there is no
CPU or PyTorch fallback, a missing library is an ImportError.
"""
from .binding import *  # noqa: F401,F403
from .binding import __all__  # noqa: F401
