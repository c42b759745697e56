"""B200-native Cassandra self-speculative decode step: CUDA library (libcass.so) plus a ctypes binding.

Importing the package loads the library; there is no CPU or PyTorch fallback for any step of the path.
"""
from . import binding  # noqa: F401
from .binding import *  # noqa: F401,F403
