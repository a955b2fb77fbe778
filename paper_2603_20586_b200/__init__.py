"""B200 (sm_100a) FastMKA attention library: Python binding of the C ABI in ``include/mka.h``.

The package holds the CUDA sources (``csrc/``), the build step (``build.py``) and the ctypes binding.
Importing it requires the built library; there is no CPU or PyTorch fallback.
"""
from .binding import *  # noqa: F401,F403
from .binding import (MkaError, lib, make_shape, mka_bwd, mka_decode, mka_decode_plan, mka_device_status,  # noqa: F401
                      mka_fwd, mka_fwd_kernel_kind, mka_fwd_tile_range, mka_router, mka_workspace_bytes, alloc_workspace, status_str)
