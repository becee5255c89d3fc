"""B200-native decode hot path of component-aware self-speculative decoding on hybrid models.

The product is the C-ABI library ``libhs.so`` (``include/hs.h``); this package is a thin ctypes
binding with the same entry points plus a small convenience class that owns the torch buffers.
"""
from .binding import (HsConfig, HsSizes, HsBuffers, HsError, lib, load_library, Engine,
                      HS_FLAG_GRAPHS, STATE_SSM, STATE_CONV, STATE_GDN, STATE_K, STATE_V, STATE_DRAFT)

__all__ = ["HsConfig", "HsSizes", "HsBuffers", "HsError", "lib", "load_library", "Engine", "HS_FLAG_GRAPHS",
           "STATE_SSM", "STATE_CONV", "STATE_GDN", "STATE_K", "STATE_V", "STATE_DRAFT"]
