"""GoodServe routing hot path on NVIDIA B200: Python binding over libgoodserve.so.

The arithmetic lives entirely in the CUDA library (``csrc/``, C ABI in
``include/goodserve.h``); this package only marshals arguments.  There is no CPU fallback:
loading fails loudly when the library is missing or no CUDA device is usable.
"""
from .binding import (NOALLOC_MAX_ACTIVE, DeviceStatus, GoodServe, GoodServeError, InstancePool,
                      library_path, load_library, risk_scan_noalloc)

__all__ = ["GoodServe", "GoodServeError", "InstancePool", "DeviceStatus", "library_path",
           "load_library", "risk_scan_noalloc", "NOALLOC_MAX_ACTIVE"]
