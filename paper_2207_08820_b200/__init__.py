"""Bit-serial ultra-low-bit convolution for NVIDIA B200 (sm_100a).

The arithmetic lives in the CUDA library behind the C ABI declared in
``include/bitserial.h``; :mod:`paper_2207_08820_b200.api` is a thin binding with the same
entry-point names.  Importing the package does not load the library; the first use of an API
name does, and raises if the library is missing (there is no CPU fallback).
"""
import importlib

_API_NAMES = ("bitpack_activations", "bitunpack_activations", "pack_weights", "bs_pack_rows",
              "bitserial_conv2d", "bitserial_gemm", "bs_check_status", "bs_popc_rate",
              "UNSIGNED", "SIGNED", "BIPOLAR", "NCHW", "NHWC")


def __getattr__(name):
    if name in _API_NAMES:
        return getattr(importlib.import_module(__name__ + ".api"), name)
    raise AttributeError(f"module {__name__!r} has no attribute {name!r}")
