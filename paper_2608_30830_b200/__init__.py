"""B200-native mover for suspended requests' paged KV cache (HBM block pool <-> pinned host DRAM).

Thin ctypes binding over libkvr.so; every step of the path runs in the CUDA
library.  There is no CPU fallback: importing `kvr` raises if the library
cannot be loaded.
"""
from . import kvr  # noqa: F401
from .kvr import KvrError, Pool, bytes_per_token  # noqa: F401
