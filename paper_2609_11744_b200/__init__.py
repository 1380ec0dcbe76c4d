"""Paged KV-cache pack / unpack and a bounded staging ring for external KV-cache
offload on NVIDIA B200: a C-ABI library (``libkvc.so``, sources in ``csrc/``,
header ``include/kvc.h``) and its ctypes binding ``kvc``."""
from . import kvc  # noqa: F401

__all__ = ["kvc"]
