"""DES-LOC fused optimizer step for NVIDIA B200: Python names for the C ABI of libdesloc.so.

``desloc_create / desloc_step / desloc_destroy`` and friends mirror include/desloc.h one to
one (see binding.py).  ``DesLoc`` is a small convenience wrapper that keeps torch tensors
alive and marshals their addresses; torch is used for device memory and streams only.
"""
from .binding import *  # noqa: F401,F403
from .binding import (DESLOC_BF16, DESLOC_F32, DTYPE_BY_NAME, OPT_BY_NAME, DeslocConfig,
                      DeslocError, make_config, ptr_array, raw_lib)
from .module import DesLoc  # noqa: F401
