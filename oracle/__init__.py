"""ctypes front end of the CPU oracle (``bitserial_oracle.c``).

TEST INFRASTRUCTURE ONLY: the tests, the smoke check and the CPU-baseline leg of
the benchmark are the only legitimate callers.  Nothing here imports the GPU
package, and the GPU package never imports this.  All arrays are numpy, all
code tensors int8 (NCHW activations, OIHW weights, row-major matrices).
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

UNSIGNED, SIGNED, BIPOLAR = 0, 1, 2

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "bitserial_oracle.c")
_SRC_FP32 = os.path.join(_HERE, "fp32_layers_oracle.c")
_SO = os.path.join(_HERE, "libbitserial_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (no fast-math, no FMA contraction) and return the .so path."""
    newest = max(os.path.getmtime(_SRC), os.path.getmtime(_SRC_FP32))
    if force or not os.path.exists(_SO) or os.path.getmtime(_SO) < newest:
        cmd = ["gcc", "-O2", "-std=c11", "-fPIC", "-shared", "-fopenmp", "-ffp-contract=off",
               "-fno-fast-math", "-o", _SO, _SRC, _SRC_FP32, "-lm"]
        subprocess.run(cmd, check=True)
    return _SO


def lib() -> ctypes.CDLL:
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
        _lib.oracle_bitserial_dot.restype = ctypes.c_int32
        _lib.oracle_bipolar_xor_dot.restype = ctypes.c_int32
        _lib.oracle_num_threads.restype = ctypes.c_int
        _lib.oracle_conv2d_i32.restype = ctypes.c_int
        _lib.oracle_gemm_i32.restype = ctypes.c_int
    return _lib


def _p(a: np.ndarray):
    return a.ctypes.data_as(ctypes.c_void_p)


def _i8(a) -> np.ndarray:
    return np.ascontiguousarray(a, dtype=np.int8)


def num_threads() -> int:
    return int(lib().oracle_num_threads())


def set_threads(n: int) -> None:
    lib().oracle_set_threads(ctypes.c_int(n))


def out_hw(H: int, W: int, R: int, S: int, stride: int, pad: int):
    return (H + 2 * pad - R) // stride + 1, (W + 2 * pad - S) // stride + 1


def quantize(x, s: float, bits: int, sign: int) -> np.ndarray:
    x = np.ascontiguousarray(x, dtype=np.float32)
    codes = np.empty(x.shape, dtype=np.int8)
    lib().oracle_quantize(_p(x), ctypes.c_long(x.size), ctypes.c_float(s), bits, sign, _p(codes))
    return codes


def dequantize(codes, s: float) -> np.ndarray:
    codes = _i8(codes)
    out = np.empty(codes.shape, dtype=np.float32)
    lib().oracle_dequantize(_p(codes), ctypes.c_long(codes.size), ctypes.c_float(s), _p(out))
    return out


def conv2d_i32(a, w, stride: int = 1, pad: int = 0) -> np.ndarray:
    a, w = _i8(a), _i8(w)
    N, C, H, W = a.shape
    O, C2, R, S = w.shape
    assert C == C2
    P, Q = out_hw(H, W, R, S, stride, pad)
    out = np.empty((N, O, P, Q), dtype=np.int32)
    rc = lib().oracle_conv2d_i32(_p(a), _p(w), N, C, H, W, O, R, S, stride, pad, _p(out))
    assert rc == 0
    return out


def gemm_i32(a, w) -> np.ndarray:
    a, w = _i8(a), _i8(w)
    M, K = a.shape
    N, K2 = w.shape
    assert K == K2
    out = np.empty((M, N), dtype=np.int32)
    lib().oracle_gemm_i32(_p(a), _p(w), M, N, K, _p(out))
    return out


def requantize(acc, scale, bias, relu: bool, out_bits: int, out_sign: int = UNSIGNED,
               res=None, res_scale: float = 0.0, channel_axis: int = 1) -> np.ndarray:
    """Epilogue on accumulators whose per-channel axis is ``channel_axis``."""
    acc = np.ascontiguousarray(acc, dtype=np.int32)
    O = acc.shape[channel_axis]
    outer = int(np.prod(acc.shape[:channel_axis], dtype=np.int64))
    inner = int(np.prod(acc.shape[channel_axis + 1:], dtype=np.int64))
    scale = np.ascontiguousarray(scale, dtype=np.float32)
    bias = np.ascontiguousarray(bias, dtype=np.float32)
    assert scale.shape == (O,) and bias.shape == (O,)
    codes = np.empty(acc.shape, dtype=np.int8)
    if res is not None:
        res = _i8(res)
        assert res.shape == acc.shape
    lib().oracle_requantize(_p(acc), ctypes.c_long(outer), O, ctypes.c_long(inner), _p(scale), _p(bias),
                            _p(res) if res is not None else None, ctypes.c_float(res_scale),
                            int(bool(relu)), out_bits, out_sign, _p(codes))
    return codes


def bitserial_dot(a, w, a_bits: int, a_sign: int, w_bits: int, w_sign: int) -> int:
    a, w = _i8(a), _i8(w)
    assert a.shape == w.shape and a.ndim == 1
    return int(lib().oracle_bitserial_dot(_p(a), _p(w), a.size, a_bits, a_sign, w_bits, w_sign))


def bipolar_xor_dot(a, w) -> int:
    a, w = _i8(a), _i8(w)
    return int(lib().oracle_bipolar_xor_dot(_p(a), _p(w), a.size))


def pack_activations(codes, bits: int, sign: int) -> np.ndarray:
    codes = _i8(codes)
    N, C, H, W = codes.shape
    out = np.empty((N, H, W, (C + 31) // 32, bits), dtype=np.uint32)
    lib().oracle_pack_activations(_p(codes), N, C, H, W, bits, sign, _p(out))
    return out


def unpack_activations(packed, C: int, bits: int, sign: int) -> np.ndarray:
    packed = np.ascontiguousarray(packed, dtype=np.uint32)
    N, H, W, Cw, b = packed.shape
    assert b == bits and Cw == (C + 31) // 32
    out = np.empty((N, C, H, W), dtype=np.int8)
    lib().oracle_unpack_activations(_p(packed), N, C, H, W, bits, sign, _p(out))
    return out


def pack_weights(codes, bits: int, sign: int) -> np.ndarray:
    codes = _i8(codes)
    O, C, R, S = codes.shape
    out = np.empty((O, R, S, (C + 31) // 32, bits), dtype=np.uint32)
    lib().oracle_pack_weights(_p(codes), O, C, R, S, bits, sign, _p(out))
    return out


def pack_rows(codes, bits: int, sign: int) -> np.ndarray:
    codes = _i8(codes)
    rows, K = codes.shape
    out = np.empty((rows, (K + 31) // 32, bits), dtype=np.uint32)
    lib().oracle_pack_rows(_p(codes), rows, K, bits, sign, _p(out))
    return out


# ---- layers kept in floating point (fp32_layers_oracle.c) -----------------------------------------------------------

def _f32(a) -> np.ndarray:
    return np.ascontiguousarray(a, dtype=np.float32)


def conv2d_f32(x, w, bias=None, stride: int = 1, pad: int = 0, relu: bool = False) -> np.ndarray:
    x, w = _f32(x), _f32(w)
    N, C, H, W = x.shape
    O, C2, R, S = w.shape
    assert C == C2
    P, Q = out_hw(H, W, R, S, stride, pad)
    out = np.empty((N, O, P, Q), dtype=np.float32)
    b = _f32(bias) if bias is not None else None
    lib().oracle_conv2d_f32(_p(x), _p(w), _p(b) if b is not None else None, N, C, H, W, O, R, S, stride, pad, int(bool(relu)), _p(out))
    return out


def maxpool2d_f32(x, k: int, stride: int, pad: int) -> np.ndarray:
    x = _f32(x)
    N, C, H, W = x.shape
    P, Q = out_hw(H, W, k, k, stride, pad)
    out = np.empty((N, C, P, Q), dtype=np.float32)
    lib().oracle_maxpool2d_f32(_p(x), N, C, H, W, k, stride, pad, _p(out))
    return out


def avgpool_codes(codes, inv: float) -> np.ndarray:
    codes = _i8(codes)
    N, C, H, W = codes.shape
    out = np.empty((N, C), dtype=np.float32)
    lib().oracle_avgpool_codes(_p(codes), N, C, H, W, ctypes.c_float(inv), _p(out))
    return out


def fc_f32(x, w, bias=None) -> np.ndarray:
    x, w = _f32(x), _f32(w)
    N, K = x.shape
    J, K2 = w.shape
    assert K == K2
    out = np.empty((N, J), dtype=np.float32)
    b = _f32(bias) if bias is not None else None
    lib().oracle_fc_f32(_p(x), _p(w), _p(b) if b is not None else None, N, K, J, _p(out))
    return out
