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


GUARD_WORDS = 64
GUARD_PATTERN = 0x5A5AA5A5


class Guarded:
    """Output buffers with guard words in front and behind: an int32 tensor of the requested shape is a view into a
    larger allocation whose first and last 64 words hold a pattern; ``check()`` asserts that no kernel touched them.
    (Stands in for a memory checker: an out-of-range store next to an output would go unseen with exact-size buffers.)"""

    def __init__(self):
        self.bufs = []

    def empty(self, shape, fill=None) -> torch.Tensor:
        n = int(np.prod(shape))
        pad = GUARD_WORDS
        raw = torch.full((n + 2 * pad,), GUARD_PATTERN, dtype=torch.int32, device="cuda")
        view = raw[pad:pad + n]
        if fill is not None:
            view.fill_(fill)
        self.bufs.append((raw, n))
        return view.view(*shape)

    def check(self) -> None:
        torch.cuda.synchronize()
        for raw, n in self.bufs:
            head = raw[:GUARD_WORDS].cpu().numpy()
            tail = raw[GUARD_WORDS + n:].cpu().numpy()
            assert (head == GUARD_PATTERN).all(), "a kernel wrote in front of an output buffer"
            assert (tail == GUARD_PATTERN).all(), "a kernel wrote behind an output buffer"


def conv_out_shapes(case, i32_layout=api.NCHW):
    N, C, H, W = case["x"].shape
    O, _, R, S = case["w"].shape
    P = (H + 2 * case["pad"] - R) // case["stride"] + 1
    Q = (W + 2 * case["pad"] - S) // case["stride"] + 1
    acc = (N, O, P, Q) if i32_layout == api.NCHW else (N, P, Q, O)
    return acc, (N, P, Q)


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
    guard = Guarded()
    acc_shape, npq = conv_out_shapes(case, i32_layout)
    out_i32 = guard.empty(acc_shape) if want_i32 else None
    if want_packed and out_packed is None:
        total = out_c_total if out_c_total else out_c_offset + case["w"].shape[0]
        out_packed = guard.empty((*npq, (total + 31) // 32, case["out_bits"]), fill=0)
    acc, packed = api.bitserial_conv2d(
        xa, wp, C=case["C"], stride=case["stride"], pad=case["pad"], a_sign=case["a_sign"], w_sign=case["w_sign"],
        scale=dev(case["scale"]) if want_packed else None, bias=dev(case["bias"]) if want_packed else None,
        relu=case["relu"], out_bits=case["out_bits"] if want_packed else 0, out_sign=case["out_sign"],
        residual=res_t, res_scale=res_scale, res_bits=res_bits, res_sign=residual[2] if residual else 0,
        res_c_offset=res_c_offset, res_c_total=res_total,
        out_i32=out_i32, i32_layout=i32_layout, out_packed=out_packed, out_c_offset=out_c_offset,
        out_c_total=out_c_total)
    api.bs_check_status()
    guard.check()
    return (acc.cpu().numpy() if acc is not None else None), (words(packed) if packed is not None else None)
