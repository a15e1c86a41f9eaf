"""Cacheback draft-and-verify step for NVIDIA B200 (sm_100a): C-ABI CUDA library + thin binding."""
from .api import Cacheback, CachebackError
from . import _lib

__all__ = ["Cacheback", "CachebackError", "_lib"]
