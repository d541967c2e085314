"""Block Transformer KV-cache attention for B200 (sm_100a): ctypes binding over libbt.so.

Importing the package loads (building first if needed) the CUDA library; there is no
CPU or framework fallback.
"""
from .binding import *  # noqa: F401,F403
from .binding import (BlockCache, BtError, LocalCache, alloc_workspace, bt_config, lib, make_config,  # noqa: F401
                      status_string)
