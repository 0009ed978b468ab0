"""Thin Python binding over the C ABI of ``include/bitserial.h``.

Argument marshalling only: tensors are torch CUDA tensors used as device buffers, streams are torch
streams, and every function forwards to the entry point of the same name.  No arithmetic of the method
happens here and nothing falls back to PyTorch ops.
"""
from __future__ import annotations

import ctypes
from typing import Optional

import torch

from ._lib import BitserialError, ConvParams, lib

UNSIGNED, SIGNED, BIPOLAR = 0, 1, 2
NCHW, NHWC = 0, 1

launch_count = 0   # kernels enqueued through this binding (every entry point below launches exactly one)


def _stream_ptr(stream: Optional[torch.cuda.Stream]) -> int:
    s = stream if stream is not None else torch.cuda.current_stream()
    return s.cuda_stream


def _ptr(t: Optional[torch.Tensor]) -> Optional[int]:
    if t is None:
        return None
    if not t.is_cuda or not t.is_contiguous():
        raise ValueError("expected a contiguous CUDA tensor")
    return t.data_ptr()


def _check(status: int, where: str) -> None:
    global launch_count
    if status != 0:
        raise BitserialError(status, where)
    launch_count += 1


def packed_act_words(N, C, H, W, bits) -> int:
    return lib().bs_packed_act_bytes(N, C, H, W, bits) // 4


def packed_wgt_words(O, C, R, S, bits) -> int:
    return lib().bs_packed_wgt_bytes(O, C, R, S, bits) // 4


def packed_rows_words(rows, K, bits) -> int:
    return lib().bs_packed_rows_bytes(rows, K, bits) // 4


def _words(n: int, device) -> torch.Tensor:
    return torch.empty(n, dtype=torch.int32, device=device)


def bitpack_activations(x: torch.Tensor, act_scale: float, a_bits: int, a_sign: int = UNSIGNED,
                        layout: int = NCHW, out: Optional[torch.Tensor] = None, stream=None) -> torch.Tensor:
    """x: float32 or int8 (codes), [N,C,H,W] (NCHW) or [N,H,W,C] (NHWC).  Returns int32 words
    viewed as [N, H, W, Cw, a_bits]."""
    if x.dtype not in (torch.float32, torch.int8):
        raise ValueError("x must be float32 or int8")
    if layout == NCHW:
        N, C, H, W = x.shape
    else:
        N, H, W, C = x.shape
    Cw = (C + 31) // 32
    if out is None:
        out = _words(N * H * W * Cw * a_bits, x.device)
    st = lib().bitpack_activations(_ptr(x), int(x.dtype == torch.float32), layout, N, C, H, W,
                                   ctypes.c_float(act_scale), a_bits, a_sign, _ptr(out), _stream_ptr(stream))
    _check(st, "bitpack_activations")
    return out.view(N, H, W, Cw, a_bits)


def bitunpack_activations(packed: torch.Tensor, C: int, a_bits: int, a_sign: int = UNSIGNED, layout: int = NCHW,
                          stream=None) -> torch.Tensor:
    N, H, W, Cw, b = packed.shape
    shape = (N, C, H, W) if layout == NCHW else (N, H, W, C)
    out = torch.empty(shape, dtype=torch.int8, device=packed.device)
    st = lib().bitunpack_activations(_ptr(packed), N, C, H, W, a_bits, a_sign, layout, _ptr(out), _stream_ptr(stream))
    _check(st, "bitunpack_activations")
    return out


def pack_weights(w_codes: torch.Tensor, w_bits: int, w_sign: int, layout: int = NCHW, stream=None) -> torch.Tensor:
    """w_codes int8 [O,C,R,S] (layout NCHW = OIHW) or [O,R,S,C].  Returns int32 words [O,R,S,Cw,w_bits]."""
    if layout == NCHW:
        O, C, R, S = w_codes.shape
    else:
        O, R, S, C = w_codes.shape
    Cw = (C + 31) // 32
    out = _words(O * R * S * Cw * w_bits, w_codes.device)
    st = lib().pack_weights(_ptr(w_codes), layout, O, C, R, S, w_bits, w_sign, _ptr(out), _stream_ptr(stream))
    _check(st, "pack_weights")
    return out.view(O, R, S, Cw, w_bits)


def bs_pack_rows(codes: torch.Tensor, bits: int, sign: int, stream=None) -> torch.Tensor:
    rows, K = codes.shape
    Kw = (K + 31) // 32
    out = _words(rows * Kw * bits, codes.device)
    st = lib().bs_pack_rows(_ptr(codes), rows, K, bits, sign, _ptr(out), _stream_ptr(stream))
    _check(st, "bs_pack_rows")
    return out.view(rows, Kw, bits)


def bitserial_conv2d(act_packed: torch.Tensor, wgt_packed: torch.Tensor, *, C: int, stride: int = 1, pad: int = 0,
                     a_sign: int = UNSIGNED, w_sign: int = SIGNED, scale: Optional[torch.Tensor] = None,
                     bias: Optional[torch.Tensor] = None, relu: bool = False, out_bits: int = 0,
                     out_sign: int = UNSIGNED, residual: Optional[torch.Tensor] = None, res_scale: float = 0.0,
                     res_bits: int = 0, res_sign: int = UNSIGNED, res_c_offset: int = 0, res_c_total: int = 0,
                     out_i32: Optional[torch.Tensor] = None, want_i32: bool = False, i32_layout: int = NCHW,
                     out_packed: Optional[torch.Tensor] = None, out_c_offset: int = 0, out_c_total: int = 0,
                     workspace: Optional[torch.Tensor] = None, wgt_tc: Optional[torch.Tensor] = None, chained: bool = False,
                     stream=None):
    """act_packed [N,H,W,Cw,a_bits], wgt_packed [O,R,S,Cw,w_bits].  Returns (out_i32 or None, out_packed or None).
    A packed output is produced when ``out_bits`` > 0 (allocated here unless ``out_packed`` is given).
    ``workspace`` (zeroed device tensor, see :func:`conv_workspace`) enables the reduction split (``bitserial_conv2d_ws``).
    ``wgt_tc`` (from :func:`tc_prepare_weights`) selects the tensor-core entry point ``bitserial_conv2d_tc``;
    with ``chained`` it is ``bitserial_conv2d_tc_chained`` (set-up overlaps the preceding kernel of the stream: filters,
    scale and bias must have been final before that kernel was launched)."""
    N, H, W, Cw, a_bits = act_packed.shape
    O, R, S, Cw2, w_bits = wgt_packed.shape
    if Cw != Cw2 or Cw != (C + 31) // 32:
        raise ValueError("channel words of activations and weights disagree")
    P = (H + 2 * pad - R) // stride + 1
    Q = (W + 2 * pad - S) // stride + 1
    dev = act_packed.device
    if want_i32 and out_i32 is None:
        shape = (N, O, P, Q) if i32_layout == NCHW else (N, P, Q, O)
        out_i32 = torch.empty(shape, dtype=torch.int32, device=dev)
    if out_bits > 0:
        if out_c_total == 0:
            out_c_total = out_c_offset + O
        if out_packed is None:
            out_packed = torch.zeros(N, P, Q, (out_c_total + 31) // 32, out_bits, dtype=torch.int32, device=dev)
    p = ConvParams(N=N, C=C, H=H, W=W, O=O, R=R, S=S, stride=stride, pad=pad, a_bits=a_bits, a_sign=a_sign,
                   w_bits=w_bits, w_sign=w_sign, scale=_ptr(scale), bias=_ptr(bias), relu=int(relu),
                   out_bits=out_bits, out_sign=out_sign, residual=_ptr(residual), res_scale=res_scale,
                   res_bits=res_bits, res_sign=res_sign, res_c_offset=res_c_offset,
                   res_c_total=res_c_total if res_c_total else res_c_offset + O,
                   out_c_offset=out_c_offset, out_c_total=out_c_total, i32_layout=i32_layout)
    if wgt_tc is not None:
        entry = lib().bitserial_conv2d_tc_chained if chained else lib().bitserial_conv2d_tc
        st = entry(_ptr(act_packed), _ptr(wgt_tc), ctypes.byref(p), _ptr(out_i32),
                   _ptr(out_packed) if out_bits > 0 else None, _stream_ptr(stream))
    elif workspace is not None:
        st = lib().bitserial_conv2d_ws(_ptr(act_packed), _ptr(wgt_packed), ctypes.byref(p), _ptr(out_i32),
                                       _ptr(out_packed) if out_bits > 0 else None, _ptr(workspace),
                                       workspace.numel() * workspace.element_size(), _stream_ptr(stream))
    else:
        st = lib().bitserial_conv2d(_ptr(act_packed), _ptr(wgt_packed), ctypes.byref(p), _ptr(out_i32),
                                    _ptr(out_packed) if out_bits > 0 else None, _stream_ptr(stream))
    _check(st, "bitserial_conv2d")
    return out_i32, (out_packed if out_bits > 0 else None)


def bitserial_gemm(a_packed: torch.Tensor, w_packed: torch.Tensor, K: int, *, a_sign: int = UNSIGNED,
                   w_sign: int = SIGNED, scale: Optional[torch.Tensor] = None, bias: Optional[torch.Tensor] = None,
                   relu: bool = False, out_bits: int = 0, out_sign: int = UNSIGNED,
                   out_i32: Optional[torch.Tensor] = None, want_i32: bool = True,
                   out_packed: Optional[torch.Tensor] = None, workspace: Optional[torch.Tensor] = None, stream=None):
    """a_packed [M,Kw,a_bits], w_packed [N,Kw,w_bits].  Returns (out_i32 [M,N] or None, out_packed or None).
    ``workspace`` (zeroed device tensor, see :func:`gemm_workspace`) enables the reduction split (``bitserial_gemm_ws``)."""
    M, Kw, a_bits = a_packed.shape
    N, Kw2, w_bits = w_packed.shape
    if Kw != Kw2 or Kw != (K + 31) // 32:
        raise ValueError("reduction words of the operands disagree")
    dev = a_packed.device
    if want_i32 and out_i32 is None:
        out_i32 = torch.empty(M, N, dtype=torch.int32, device=dev)
    if out_bits > 0 and out_packed is None:
        out_packed = torch.zeros(M, (N + 31) // 32, out_bits, dtype=torch.int32, device=dev)
    if workspace is not None:
        st = lib().bitserial_gemm_ws(_ptr(a_packed), _ptr(w_packed), M, N, K, a_bits, a_sign, w_bits, w_sign,
                                     _ptr(scale), _ptr(bias), int(relu), out_bits, out_sign, _ptr(out_i32),
                                     _ptr(out_packed) if out_bits > 0 else None, _ptr(workspace),
                                     workspace.numel() * workspace.element_size(), _stream_ptr(stream))
    else:
        st = lib().bitserial_gemm(_ptr(a_packed), _ptr(w_packed), M, N, K, a_bits, a_sign, w_bits, w_sign,
                                  _ptr(scale), _ptr(bias), int(relu), out_bits, out_sign, _ptr(out_i32),
                                  _ptr(out_packed) if out_bits > 0 else None, _stream_ptr(stream))
    _check(st, "bitserial_gemm")
    return out_i32, (out_packed if out_bits > 0 else None)


def tc_prepare_weights(wgt_packed: torch.Tensor, C: int, w_sign: int, a_bits: int, stream=None) -> torch.Tensor:
    """Packed weights [O,R,S,Cw,w_bits] -> int8 filter tiles for the tensor-core entry points."""
    O, R, S, Cw, w_bits = wgt_packed.shape
    nbytes = lib().bs_tc_weights_bytes(O, C, R, S)
    if nbytes == 0:
        raise BitserialError(2, "bs_tc_weights_bytes")
    out = torch.empty(nbytes, dtype=torch.int8, device=wgt_packed.device)
    st = lib().bs_tc_prepare_weights(_ptr(wgt_packed), O, C, R, S, w_bits, w_sign, a_bits, _ptr(out), _stream_ptr(stream))
    _check(st, "bs_tc_prepare_weights")
    return out


def tc_supported(N, C, H, W, O, k, stride, pad, a_bits, a_sign, w_bits, w_sign) -> bool:
    p = ConvParams(N=N, C=C, H=H, W=W, O=O, R=k, S=k, stride=stride, pad=pad, a_bits=a_bits, a_sign=a_sign,
                   w_bits=w_bits, w_sign=w_sign)
    return bool(lib().bs_tc_supported(ctypes.byref(p)))


def conv_params(act_shape, wgt_shape, *, C: int, stride: int = 1, pad: int = 0, a_sign: int = UNSIGNED, w_sign: int = SIGNED,
                scale: Optional[torch.Tensor] = None, bias: Optional[torch.Tensor] = None, relu: bool = False, out_bits: int = 0,
                out_sign: int = UNSIGNED, residual: Optional[torch.Tensor] = None, res_scale: float = 0.0, res_bits: int = 0,
                res_sign: int = UNSIGNED) -> ConvParams:
    """``bs_conv_params`` of a layer whose packed output is a whole tensor (no channel offset), from the shapes of the packed
    operands; for :func:`tc_chain_workspace_bytes` and :func:`bitserial_conv2d_tc_chain`."""
    N, H, W, Cw, a_bits = act_shape
    O, R, S, Cw2, w_bits = wgt_shape
    if Cw != Cw2 or Cw != (C + 31) // 32:
        raise ValueError("channel words of activations and weights disagree")
    return ConvParams(N=N, C=C, H=H, W=W, O=O, R=R, S=S, stride=stride, pad=pad, a_bits=a_bits, a_sign=a_sign, w_bits=w_bits,
                      w_sign=w_sign, scale=_ptr(scale), bias=_ptr(bias), relu=int(relu), out_bits=out_bits, out_sign=out_sign,
                      residual=_ptr(residual), res_scale=res_scale, res_bits=res_bits, res_sign=res_sign, res_c_offset=0,
                      res_c_total=O, out_c_offset=0, out_c_total=O, i32_layout=NCHW)


def _params_array(params):
    arr = (ConvParams * len(params))()
    for k, q in enumerate(params):
        ctypes.memmove(ctypes.addressof(arr[k]), ctypes.addressof(q), ctypes.sizeof(ConvParams))
    return arr


def tc_chain_workspace_bytes(params) -> int:
    """Bytes of the (zero-filled) workspace ``bitserial_conv2d_tc_chain`` needs for these layers; 0 when they cannot run as
    one launch."""
    return int(lib().bs_tc_chain_workspace_bytes(_params_array(params), len(params)))


def bitserial_conv2d_tc_chain(acts, wgts_tc, params, outs, workspace: torch.Tensor, chained: bool = False, stream=None) -> None:
    """Several same-shaped layers in one launch (``bitserial_conv2d_tc_chain``): per layer the packed input, the prepared
    filters, the :func:`conv_params` and the packed output tensor.  ``workspace``: device tensor of
    :func:`tc_chain_workspace_bytes` bytes, zero-filled once before its first use."""
    n = len(params)
    vp = ctypes.c_void_p * n
    st = lib().bitserial_conv2d_tc_chain(n, vp(*[_ptr(t) for t in acts]), vp(*[_ptr(t) for t in wgts_tc]), _params_array(params),
                                         vp(*[_ptr(t) for t in outs]), _ptr(workspace), workspace.numel() * workspace.element_size(),
                                         int(chained), _stream_ptr(stream))
    _check(st, "bitserial_conv2d_tc_chain")


def bitserial_gemm_tc(a_packed: torch.Tensor, w_tc: torch.Tensor, N: int, K: int, w_bits: int, *, a_sign: int = UNSIGNED,
                      w_sign: int = SIGNED, scale=None, bias=None, relu: bool = False, out_bits: int = 0,
                      out_sign: int = UNSIGNED, want_i32: bool = True, out_i32: Optional[torch.Tensor] = None,
                      out_packed: Optional[torch.Tensor] = None, stream=None):
    """Tensor-core matrix product: a_packed [M,Kw,a_bits], w_tc from tc_prepare_weights on the [N,1,1,Kw,w_bits] rows."""
    M, Kw, a_bits = a_packed.shape
    dev = a_packed.device
    if want_i32 and out_i32 is None:
        out_i32 = torch.empty(M, N, dtype=torch.int32, device=dev)
    if out_bits > 0 and out_packed is None:
        out_packed = torch.zeros(M, (N + 31) // 32, out_bits, dtype=torch.int32, device=dev)
    if out_bits <= 0:
        out_packed = None
    st = lib().bitserial_gemm_tc(_ptr(a_packed), _ptr(w_tc), M, N, K, a_bits, a_sign, w_bits, w_sign, _ptr(scale), _ptr(bias),
                                 int(relu), out_bits, out_sign, _ptr(out_i32), _ptr(out_packed), _stream_ptr(stream))
    _check(st, "bitserial_gemm_tc")
    return out_i32, out_packed


def gemm_workspace(M: int, N: int, K: int, a_bits: int, a_sign: int, w_bits: int, w_sign: int, device="cuda"):
    """Zeroed workspace for the reduction split of this matrix product, or None when the planner would not split."""
    nbytes = lib().bs_gemm_workspace_bytes(M, N, K, a_bits, a_sign, w_bits, w_sign)
    return torch.zeros((nbytes + 3) // 4, dtype=torch.int32, device=device) if nbytes else None


def conv_workspace(N: int, C: int, H: int, W: int, O: int, k: int, stride: int, pad: int, a_bits: int, a_sign: int,
                   w_bits: int, w_sign: int, device="cuda"):
    """Zeroed workspace for the reduction split of this convolution, or None when the planner would not split."""
    p = ConvParams(N=N, C=C, H=H, W=W, O=O, R=k, S=k, stride=stride, pad=pad, a_bits=a_bits, a_sign=a_sign,
                   w_bits=w_bits, w_sign=w_sign)
    nbytes = lib().bs_conv_workspace_bytes(ctypes.byref(p))
    return torch.zeros((nbytes + 3) // 4, dtype=torch.int32, device=device) if nbytes else None


def conv2d_f32(x: torch.Tensor, w: torch.Tensor, bias: Optional[torch.Tensor] = None, stride: int = 1, pad: int = 0, relu: bool = False,
               out: Optional[torch.Tensor] = None, stream=None) -> torch.Tensor:
    """Floating-point convolution of the layers kept in FP32 (``bs_conv2d_f32``): x [N,C,H,W], w [O,C,R,S] float32."""
    N, C, H, W = x.shape
    O, C2, R, S = w.shape
    if C != C2 or x.dtype != torch.float32 or w.dtype != torch.float32:
        raise ValueError("float32 tensors with matching channels expected")
    P, Q = (H + 2 * pad - R) // stride + 1, (W + 2 * pad - S) // stride + 1
    if out is None:
        out = torch.empty(N, O, P, Q, dtype=torch.float32, device=x.device)
    _check(lib().bs_conv2d_f32(_ptr(x), _ptr(w), _ptr(bias), N, C, H, W, O, R, S, stride, pad, int(relu), _ptr(out), _stream_ptr(stream)),
           "bs_conv2d_f32")
    return out


def maxpool2d_f32(x: torch.Tensor, k: int, stride: int, pad: int, out: Optional[torch.Tensor] = None, stream=None) -> torch.Tensor:
    N, C, H, W = x.shape
    P, Q = (H + 2 * pad - k) // stride + 1, (W + 2 * pad - k) // stride + 1
    if out is None:
        out = torch.empty(N, C, P, Q, dtype=torch.float32, device=x.device)
    _check(lib().bs_maxpool2d_f32(_ptr(x), N, C, H, W, k, stride, pad, _ptr(out), _stream_ptr(stream)), "bs_maxpool2d_f32")
    return out


def avgpool_codes_f32(packed: torch.Tensor, C: int, a_sign: int, inv: float, out: Optional[torch.Tensor] = None, stream=None) -> torch.Tensor:
    """Global average pool of packed codes [N,H,W,Cw,a_bits] -> float32 [N,C] (``bs_avgpool_codes_f32``)."""
    N, H, W, Cw, a_bits = packed.shape
    if out is None:
        out = torch.empty(N, C, dtype=torch.float32, device=packed.device)
    _check(lib().bs_avgpool_codes_f32(_ptr(packed), N, C, H, W, a_bits, a_sign, ctypes.c_float(inv), _ptr(out), _stream_ptr(stream)),
           "bs_avgpool_codes_f32")
    return out


def fc_f32(x: torch.Tensor, w: torch.Tensor, bias: Optional[torch.Tensor] = None, out: Optional[torch.Tensor] = None, stream=None) -> torch.Tensor:
    N, K = x.shape
    J, K2 = w.shape
    if K != K2:
        raise ValueError("inner dimensions disagree")
    if out is None:
        out = torch.empty(N, J, dtype=torch.float32, device=x.device)
    _check(lib().bs_fc_f32(_ptr(x), _ptr(w), _ptr(bias), N, K, J, _ptr(out), _stream_ptr(stream)), "bs_fc_f32")
    return out


def bs_check_status(stream=None) -> None:
    st = lib().bs_check_status(_stream_ptr(stream))
    if st != 0:
        raise BitserialError(st, "bs_check_status")


def selftest_wait_timeout(polls: int = 256, stream=None) -> None:
    """Launches the kernel whose bounded wait runs out (``bs_selftest_wait_timeout``); the next :func:`bs_check_status`
    raises ``BitserialError`` with BS_ERR_TIMEOUT once."""
    _check(lib().bs_selftest_wait_timeout(int(polls), _stream_ptr(stream)), "bs_selftest_wait_timeout")


def l2_prefetch(tensors, stream=None) -> None:
    """Hint: bring the given device tensors into L2 while the following kernels of the stream run (``bs_l2_prefetch``)."""
    ts = [t for t in tensors if t is not None and t.numel() > 0]
    if not ts:
        return
    ptrs = (ctypes.c_void_p * len(ts))(*[t.data_ptr() for t in ts])
    sizes = (ctypes.c_size_t * len(ts))(*[t.numel() * t.element_size() for t in ts])
    _check(lib().bs_l2_prefetch(ptrs, sizes, len(ts), _stream_ptr(stream)), "bs_l2_prefetch")


def bs_popc_rate(iters: int = 4096) -> float:
    out = ctypes.c_double(0.0)
    st = lib().bs_popc_rate(iters, ctypes.byref(out))
    if st != 0:
        raise BitserialError(st, "bs_popc_rate")
    return out.value
