"""Helpers shared by the GPU parity tests: move seeded numpy inputs to the device, call the C ABI
through the binding, bring results back as numpy for element-by-element comparison with the oracle."""
import numpy as np
import torch

from paper_2207_08820_b200 import api


def dev(a: np.ndarray) -> torch.Tensor:
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def words(t: torch.Tensor) -> np.ndarray:
    """int32 device words -> uint32 numpy."""
    return t.cpu().numpy().view(np.uint32)


def gpu_conv(case, want_i32=True, want_packed=True, i32_layout=api.NCHW, residual=None, res_scale=0.0,
             out_c_offset=0, out_c_total=0, out_packed=None, res_c_offset=0):
    """Runs pack -> conv for a workloads.single_conv_case-style dict.  Returns (acc NCHW/NHWC numpy or None,
    packed output words numpy or None)."""
    x = dev(case["x"])
    w = dev(case["w"])
    xa = api.bitpack_activations(x, 1.0, case["a_bits"], case["a_sign"], api.NCHW)
    wp = api.pack_weights(w, case["w_bits"], case["w_sign"], api.NCHW)
    res_t = None
    res_bits = 0
    res_total = 0
    if residual is not None:
        res_codes, res_bits, res_sign = residual
        res_total = res_codes.shape[1]
        res_t = api.bitpack_activations(dev(res_codes), 1.0, res_bits, res_sign, api.NCHW)
    acc, packed = api.bitserial_conv2d(
        xa, wp, C=case["C"], stride=case["stride"], pad=case["pad"], a_sign=case["a_sign"], w_sign=case["w_sign"],
        scale=dev(case["scale"]) if want_packed else None, bias=dev(case["bias"]) if want_packed else None,
        relu=case["relu"], out_bits=case["out_bits"] if want_packed else 0, out_sign=case["out_sign"],
        residual=res_t, res_scale=res_scale, res_bits=res_bits, res_sign=residual[2] if residual else 0,
        res_c_offset=res_c_offset, res_c_total=res_total,
        want_i32=want_i32, i32_layout=i32_layout, out_packed=out_packed, out_c_offset=out_c_offset,
        out_c_total=out_c_total)
    api.bs_check_status()
    return (acc.cpu().numpy() if acc is not None else None), (words(packed) if packed is not None else None)
