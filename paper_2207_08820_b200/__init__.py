"""Bit-serial ultra-low-bit convolution for NVIDIA B200 (sm_100a).

The arithmetic lives in the CUDA library behind the C ABI declared in
``include/bitserial.h``; :mod:`paper_2207_08820_b200.api` is a thin binding with the same
entry-point names.  Importing the package does not load the library; the first use of an API
name does, and raises if the library is missing (there is no CPU fallback).
"""
_API_MODULE = None


def __getattr__(name):
    if name.startswith("__"):
        raise AttributeError(name)
    global _API_MODULE
    if _API_MODULE is None:
        from . import api as _api
        _API_MODULE = _api
    try:
        return getattr(_API_MODULE, name)
    except AttributeError:
        raise AttributeError(f"module 'paper_2207_08820_b200' has no attribute {name!r}") from None
