"""Cacheback draft-and-verify step for NVIDIA B200 (sm_100a): C-ABI CUDA library + thin binding."""
from .api import Cacheback, CachebackError, FrozenTable, cb_accept_static
from . import _lib

__all__ = ["Cacheback", "CachebackError", "FrozenTable", "cb_accept_static", "_lib"]
