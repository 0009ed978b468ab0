"""Loads the CUDA library.  There is no fallback: a missing library is an error."""
from __future__ import annotations

import ctypes
import os

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libbitserial_b200.so")
_lib = None


class BitserialError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        name = lib().bs_status_string(status).decode() if _lib is not None else str(status)
        super().__init__(f"{where} failed: {name} ({status})")


class ConvParams(ctypes.Structure):
    """Mirror of ``bs_conv_params`` (include/bitserial.h)."""
    _fields_ = [
        ("N", ctypes.c_int), ("C", ctypes.c_int), ("H", ctypes.c_int), ("W", ctypes.c_int),
        ("O", ctypes.c_int), ("R", ctypes.c_int), ("S", ctypes.c_int),
        ("stride", ctypes.c_int), ("pad", ctypes.c_int),
        ("a_bits", ctypes.c_int), ("a_sign", ctypes.c_int),
        ("w_bits", ctypes.c_int), ("w_sign", ctypes.c_int),
        ("scale", ctypes.c_void_p), ("bias", ctypes.c_void_p),
        ("relu", ctypes.c_int),
        ("out_bits", ctypes.c_int), ("out_sign", ctypes.c_int),
        ("residual", ctypes.c_void_p), ("res_scale", ctypes.c_float),
        ("res_bits", ctypes.c_int), ("res_sign", ctypes.c_int),
        ("res_c_offset", ctypes.c_int), ("res_c_total", ctypes.c_int),
        ("out_c_offset", ctypes.c_int), ("out_c_total", ctypes.c_int),
        ("i32_layout", ctypes.c_int),
    ]


def lib() -> ctypes.CDLL:
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise ImportError(
            f"{LIB_PATH} is missing: build it with `python -m paper_2207_08820_b200.build` "
            "(nvcc, sm_100a).  This library has no CPU or PyTorch fallback.")
    L = ctypes.CDLL(LIB_PATH)
    vp, i, f = ctypes.c_void_p, ctypes.c_int, ctypes.c_float
    L.bs_packed_act_bytes.restype = ctypes.c_size_t
    L.bs_packed_act_bytes.argtypes = [i] * 5
    L.bs_packed_wgt_bytes.restype = ctypes.c_size_t
    L.bs_packed_wgt_bytes.argtypes = [i] * 5
    L.bs_packed_rows_bytes.restype = ctypes.c_size_t
    L.bs_packed_rows_bytes.argtypes = [i] * 3
    L.bitpack_activations.restype = i
    L.bitpack_activations.argtypes = [vp, i, i, i, i, i, i, f, i, i, vp, vp]
    L.bitunpack_activations.restype = i
    L.bitunpack_activations.argtypes = [vp, i, i, i, i, i, i, i, vp, vp]
    L.pack_weights.restype = i
    L.pack_weights.argtypes = [vp, i, i, i, i, i, i, i, vp, vp]
    L.bs_pack_rows.restype = i
    L.bs_pack_rows.argtypes = [vp, i, i, i, i, vp, vp]
    L.bitserial_conv2d.restype = i
    L.bitserial_conv2d.argtypes = [vp, vp, ctypes.POINTER(ConvParams), vp, vp, vp]
    L.bitserial_gemm.restype = i
    L.bitserial_gemm.argtypes = [vp, vp, i, i, i, i, i, i, i, vp, vp, i, i, i, vp, vp, vp]
    L.bitserial_conv2d_ws.restype = i
    L.bitserial_conv2d_ws.argtypes = [vp, vp, ctypes.POINTER(ConvParams), vp, vp, vp, ctypes.c_size_t, vp]
    L.bitserial_gemm_ws.restype = i
    L.bitserial_gemm_ws.argtypes = [vp, vp, i, i, i, i, i, i, i, vp, vp, i, i, i, vp, vp, vp, ctypes.c_size_t, vp]
    L.bs_conv_workspace_bytes.restype = ctypes.c_size_t
    L.bs_conv_workspace_bytes.argtypes = [ctypes.POINTER(ConvParams)]
    L.bs_gemm_workspace_bytes.restype = ctypes.c_size_t
    L.bs_gemm_workspace_bytes.argtypes = [i] * 7
    L.bitserial_gemm_noalloc.restype = i
    L.bitserial_gemm_noalloc.argtypes = [vp, vp, i, i, i, i, i, i, i, vp, vp, i, i, i, vp, vp, vp]
    L.bs_gemm_noalloc_max_scratch_bytes.restype = ctypes.c_size_t
    L.bs_gemm_noalloc_max_scratch_bytes.argtypes = []
    L.bs_selftest_dirty_noalloc_scratch.restype = i
    L.bs_selftest_dirty_noalloc_scratch.argtypes = [i, vp]
    L.bs_tc_weights_bytes.restype = ctypes.c_size_t
    L.bs_tc_weights_bytes.argtypes = [i] * 4
    L.bs_tc_prepare_weights.restype = i
    L.bs_tc_prepare_weights.argtypes = [vp, i, i, i, i, i, i, i, vp, vp]
    L.bs_tc_supported.restype = i
    L.bs_tc_supported.argtypes = [ctypes.POINTER(ConvParams)]
    L.bitserial_conv2d_tc.restype = i
    L.bitserial_conv2d_tc.argtypes = [vp, vp, ctypes.POINTER(ConvParams), vp, vp, vp]
    L.bs_l2_prefetch.restype = i
    L.bs_l2_prefetch.argtypes = [ctypes.POINTER(ctypes.c_void_p), ctypes.POINTER(ctypes.c_size_t), ctypes.c_int, vp]
    L.bitserial_conv2d_tc_chained.restype = i
    L.bitserial_conv2d_tc_chained.argtypes = [vp, vp, ctypes.POINTER(ConvParams), vp, vp, vp]
    L.bs_tc_chain_workspace_bytes.restype = ctypes.c_size_t
    L.bs_tc_chain_workspace_bytes.argtypes = [ctypes.POINTER(ConvParams), i]
    L.bitserial_conv2d_tc_chain.restype = i
    L.bitserial_conv2d_tc_chain.argtypes = [i, ctypes.POINTER(ctypes.c_void_p), ctypes.POINTER(ctypes.c_void_p), ctypes.POINTER(ConvParams),
                                            ctypes.POINTER(ctypes.c_void_p), vp, ctypes.c_size_t, i, vp]
    L.bitserial_gemm_tc.restype = i
    L.bitserial_gemm_tc.argtypes = [vp, vp, i, i, i, i, i, i, i, vp, vp, i, i, i, vp, vp, vp]
    L.bs_conv2d_f32.restype = i
    L.bs_conv2d_f32.argtypes = [vp, vp, vp, i, i, i, i, i, i, i, i, i, i, vp, vp]
    L.bs_maxpool2d_f32.restype = i
    L.bs_maxpool2d_f32.argtypes = [vp, i, i, i, i, i, i, i, vp, vp]
    L.bs_avgpool_codes_f32.restype = i
    L.bs_avgpool_codes_f32.argtypes = [vp, i, i, i, i, i, i, ctypes.c_float, vp, vp]
    L.bs_fc_f32.restype = i
    L.bs_fc_f32.argtypes = [vp, vp, vp, i, i, i, vp, vp]
    L.bs_check_status.restype = i
    L.bs_check_status.argtypes = [vp]
    L.bs_quantiser_bounds.restype = i
    L.bs_quantiser_bounds.argtypes = [ctypes.c_float, i, i, ctypes.POINTER(ctypes.c_float)]
    L.bs_requant_bounds.restype = i
    L.bs_requant_bounds.argtypes = [i, ctypes.c_float, i, i, i, i, i, ctypes.POINTER(ctypes.c_float)]
    L.bs_selftest_wait_timeout.restype = i
    L.bs_selftest_wait_timeout.argtypes = [i, vp]
    L.bs_popc_rate.restype = i
    L.bs_popc_rate.argtypes = [i, ctypes.POINTER(ctypes.c_double)]
    L.bs_status_string.restype = ctypes.c_char_p
    L.bs_status_string.argtypes = [i]
    _lib = L
    return L


EXPORTED = ("bs_packed_act_bytes", "bs_packed_wgt_bytes", "bs_packed_rows_bytes", "bitpack_activations",
            "bitunpack_activations", "pack_weights", "bs_pack_rows", "bitserial_conv2d", "bitserial_gemm",
            "bitserial_conv2d_ws", "bitserial_gemm_ws", "bs_conv_workspace_bytes", "bs_gemm_workspace_bytes",
            "bitserial_gemm_noalloc", "bs_gemm_noalloc_max_scratch_bytes", "bs_selftest_dirty_noalloc_scratch",
            "bs_tc_weights_bytes", "bs_tc_prepare_weights", "bs_tc_supported", "bitserial_conv2d_tc", "bitserial_conv2d_tc_chained", "bs_tc_chain_workspace_bytes", "bitserial_conv2d_tc_chain", "bitserial_gemm_tc", "bs_l2_prefetch",
            "bs_conv2d_f32", "bs_maxpool2d_f32", "bs_avgpool_codes_f32", "bs_fc_f32",
            "bs_check_status", "bs_quantiser_bounds", "bs_requant_bounds", "bs_selftest_wait_timeout", "bs_popc_rate", "bs_status_string")
