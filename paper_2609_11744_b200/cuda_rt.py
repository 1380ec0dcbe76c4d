"""Minimal ctypes access to the CUDA runtime for callers that hold raw addresses
(ring slots are raw pointers): asynchronous memcpy between host and device."""
from __future__ import annotations

import ctypes

H2H, H2D, D2H, D2D = 0, 1, 2, 3
_rt = None


def _cudart():
    global _rt
    if _rt is None:
        last = None
        for name in ("libcudart.so.12", "libcudart.so", "/usr/local/cuda/lib64/libcudart.so"):
            try:
                _rt = ctypes.CDLL(name)
                break
            except OSError as e:  # try the next name
                last = e
        if _rt is None:
            raise ImportError("CUDA runtime library not found: %s" % last)
        _rt.cudaMemcpyAsync.restype = ctypes.c_int
        _rt.cudaMemcpyAsync.argtypes = [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_size_t,
                                        ctypes.c_int, ctypes.c_void_p]
    return _rt


def memcpy_async(dst: int, src: int, nbytes: int, kind: int, stream) -> None:
    """cudaMemcpyAsync on raw addresses; ``stream`` is a torch stream or a raw handle."""
    s = stream if isinstance(stream, int) else int(stream.cuda_stream)
    rc = _cudart().cudaMemcpyAsync(dst, src, nbytes, kind, s)
    if rc != 0:
        raise RuntimeError("cudaMemcpyAsync failed with error %d" % rc)
