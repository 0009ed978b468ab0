"""Seeded random-shape sweep: shapes, bit-widths, signs, strides and pads drawn within the library's limits, on the
popcount entry point and, where the shape is supported, on the tensor-core entry point.  Accumulators bit-exact against
the oracle's direct integer convolution / matrix product, requantised codes equal to the oracle's epilogue and plane
split (tolerance: at most 1e-4 of codes off by one level; zero expected)."""
import numpy as np
import pytest

import oracle
from paper_2207_08820_b200 import api, workloads as wl
from gpu_util import Guarded, conv_out_shapes, dev, gpu_conv, words

pytestmark = pytest.mark.gpu


def draw_conv(rng):
    k = int(rng.choice([1, 3, 3, 5, 7]))
    stride = int(rng.choice([1, 2]))
    pad = int(rng.integers(0, k // 2 + 1))
    a_bits = int(rng.integers(1, 5))
    w_bits = int(rng.integers(1, 5))
    a_sign = int(rng.choice([0, 0, 1])) if a_bits > 1 else int(rng.choice([0, 2]))
    if a_sign == 2:
        pad = 0                                    # zero padding is not representable in {-1, +1}
    w_sign = (int(rng.choice([0, 1])) if w_bits > 1 else int(rng.choice([0, 2])))
    H = int(rng.integers(max(k - 2 * pad, 1), 24))
    W = int(rng.integers(max(k - 2 * pad, 1), 24))
    C = int(rng.choice([32, 33, 40, 64, 64, 70, 96, 128, 160]))
    O = int(rng.choice([8, 24, 32, 40, 64, 72, 96, 128, 130]))
    N = int(rng.integers(1, 4))
    out_bits = int(rng.integers(1, 5))
    return dict(N=N, C=C, H=H, W=W, O=O, k=k, stride=stride, pad=pad, a_bits=a_bits, a_sign=a_sign, w_bits=w_bits,
                w_sign=w_sign, out_bits=out_bits)


@pytest.mark.parametrize("index", range(48))
def test_random_conv_shape(index):
    rng = np.random.default_rng(90000 + index)
    d = draw_conv(rng)
    c = wl.single_conv_case(seed=91000 + index, calibrated=True, **d)
    want = oracle.conv2d_i32(c["x"], c["w"], d["stride"], d["pad"])
    codes = oracle.requantize(want, c["scale"], c["bias"], True, d["out_bits"], 0)
    want_packed = oracle.pack_activations(codes, d["out_bits"], 0)
    acc, packed = gpu_conv(c)                      # popcount entry point, guard words around both outputs
    assert np.array_equal(acc, want), d
    assert np.array_equal(packed, want_packed), d
    if api.tc_supported(d["N"], d["C"], d["H"], d["W"], d["O"], d["k"], d["stride"], d["pad"], d["a_bits"], d["a_sign"],
                        d["w_bits"], d["w_sign"]):
        xa = api.bitpack_activations(dev(c["x"]), 1.0, d["a_bits"], d["a_sign"], api.NCHW)
        wp = api.pack_weights(dev(c["w"]), d["w_bits"], d["w_sign"], api.NCHW)
        wt = api.tc_prepare_weights(wp, d["C"], d["w_sign"], d["a_bits"])
        guard = Guarded()
        acc_shape, npq = conv_out_shapes(c)
        a2, p2 = api.bitserial_conv2d(xa, wp, C=d["C"], stride=d["stride"], pad=d["pad"], a_sign=d["a_sign"], w_sign=d["w_sign"],
                                      scale=dev(c["scale"]), bias=dev(c["bias"]), relu=True, out_bits=d["out_bits"],
                                      out_i32=guard.empty(acc_shape),
                                      out_packed=guard.empty((*npq, (d["O"] + 31) // 32, d["out_bits"]), fill=0), wgt_tc=wt)
        api.bs_check_status()
        guard.check()
        assert np.array_equal(a2.cpu().numpy(), want), d
        assert np.array_equal(words(p2), want_packed), d


@pytest.mark.parametrize("index", range(16))
def test_random_gemm_shape(index):
    rng = np.random.default_rng(92000 + index)
    M, N, K = int(rng.integers(1, 400)), int(rng.integers(1, 300)), int(rng.integers(1, 1500))
    a_bits, w_bits = int(rng.integers(1, 5)), int(rng.integers(1, 5))
    a_sign = int(rng.choice([0, 1])) if a_bits > 1 else int(rng.choice([0, 2]))
    w_sign = int(rng.choice([0, 1])) if w_bits > 1 else int(rng.choice([0, 2]))
    c = wl.gemm_case(M, N, K, seed=93000 + index, a_bits=a_bits, a_sign=a_sign, w_bits=w_bits, w_sign=w_sign)
    guard = Guarded()
    out, _ = api.bitserial_gemm(api.bs_pack_rows(dev(c["a"]), a_bits, a_sign), api.bs_pack_rows(dev(c["w"]), w_bits, w_sign), K,
                                a_sign=a_sign, w_sign=w_sign, out_i32=guard.empty((M, N)))
    api.bs_check_status()
    guard.check()
    assert np.array_equal(out.cpu().numpy(), oracle.gemm_i32(c["a"], c["w"])), (M, N, K, a_bits, a_sign, w_bits, w_sign)
