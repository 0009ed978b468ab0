"""GPU parity for the tensor-core entry points: int32 accumulators bit-exact against the oracle's direct integer
convolution, requantised codes equal to the oracle's epilogue (tolerance: at most 1e-4 of codes off by one level;
zero expected), and identical to the popcount entry points."""
import numpy as np
import pytest
import torch

import oracle
from paper_2207_08820_b200 import api, workloads as wl
from gpu_util import Guarded, conv_out_shapes, dev, words

pytestmark = pytest.mark.gpu


def run_tc(c, residual=None, res_scale=0.0, want_packed=True, i32_layout=api.NCHW):
    xa = api.bitpack_activations(dev(c["x"]), 1.0, c["a_bits"], c["a_sign"], api.NCHW)
    wp = api.pack_weights(dev(c["w"]), c["w_bits"], c["w_sign"], api.NCHW)
    wt = api.tc_prepare_weights(wp, c["C"], c["w_sign"], c["a_bits"])
    res_t, res_total = None, 0
    if residual is not None:
        res_t = api.bitpack_activations(dev(residual), 1.0, 2, 0, api.NCHW)
        res_total = residual.shape[1]
    guard = Guarded()                      # guard words around both outputs, checked after the call
    acc_shape, npq = conv_out_shapes(c, i32_layout)
    out_i32 = guard.empty(acc_shape)
    out_packed = guard.empty((*npq, (c["w"].shape[0] + 31) // 32, c["out_bits"]), fill=0) if want_packed else None
    acc, packed = api.bitserial_conv2d(
        xa, wp, C=c["C"], stride=c["stride"], pad=c["pad"], a_sign=c["a_sign"], w_sign=c["w_sign"],
        scale=dev(c["scale"]) if want_packed else None, bias=dev(c["bias"]) if want_packed else None, relu=c["relu"],
        out_bits=c["out_bits"] if want_packed else 0, out_sign=0, residual=res_t, res_scale=res_scale,
        res_bits=2 if residual is not None else 0, res_c_total=res_total, out_i32=out_i32, out_packed=out_packed,
        i32_layout=i32_layout, wgt_tc=wt)
    api.bs_check_status()
    guard.check()
    return acc.cpu().numpy(), (words(packed) if packed is not None else None)


@pytest.mark.parametrize("k,stride,pad", [(1, 1, 0), (1, 2, 0), (3, 1, 1), (3, 2, 1), (3, 1, 0), (3, 2, 0), (5, 1, 2), (7, 2, 3)])
@pytest.mark.parametrize("hw", [(7, 7), (14, 14), (9, 20), (23, 11), (56, 56)])
def test_tc_conv_geometry(k, stride, pad, hw):
    H, W = hw
    if H + 2 * pad < k or W + 2 * pad < k:
        pytest.skip("kernel larger than padded image")
    c = wl.single_conv_case(seed=k * 100 + stride * 10 + pad + H, N=3, C=64, H=H, W=W, O=40, k=k, stride=stride, pad=pad,
                            calibrated=True)
    acc, packed = run_tc(c)
    want = oracle.conv2d_i32(c["x"], c["w"], stride, pad)
    assert np.array_equal(acc, want)
    codes = oracle.requantize(want, c["scale"], c["bias"], True, 2, 0)
    assert np.array_equal(packed, oracle.pack_activations(codes, 2, 0))


@pytest.mark.parametrize("ab,asg,C", [(2, 0, 64), (2, 1, 128), (4, 0, 32), (4, 1, 96), (1, 0, 128), (3, 0, 128), (1, 2, 128)])
@pytest.mark.parametrize("wb,wsg", [(1, 2), (2, 1), (3, 1), (4, 1), (2, 0)])
def test_tc_bitwidths_and_signs(ab, asg, C, wb, wsg):
    pad = 0 if asg == 2 else 1
    c = wl.single_conv_case(seed=ab * 10 + wb, N=2, C=C, H=12, W=10, O=72, pad=pad, a_bits=ab, a_sign=asg, w_bits=wb, w_sign=wsg,
                            out_bits=2, calibrated=True)
    acc, packed = run_tc(c, i32_layout=api.NHWC)
    want = oracle.conv2d_i32(c["x"], c["w"], 1, pad)
    assert np.array_equal(acc, want.transpose(0, 2, 3, 1))
    codes = oracle.requantize(want, c["scale"], c["bias"], True, 2, 0)
    assert np.array_equal(packed, oracle.pack_activations(codes, 2, 0))


@pytest.mark.parametrize("C,O", [(64, 32), (64, 128), (128, 64), (256, 96), (512, 64), (192, 200)])
def test_tc_channel_counts_multi_chunk(C, O):
    c = wl.single_conv_case(seed=C + O, N=2, C=C, H=14, W=14, O=O, calibrated=True)
    acc, packed = run_tc(c)
    want = oracle.conv2d_i32(c["x"], c["w"], 1, 1)
    assert np.array_equal(acc, want)
    codes = oracle.requantize(want, c["scale"], c["bias"], True, 2, 0)
    assert np.array_equal(packed, oracle.pack_activations(codes, 2, 0))


@pytest.mark.parametrize("k,stride,pad", [(1, 1, 0), (3, 1, 1), (3, 2, 1), (1, 2, 0), (3, 1, 0)])
def test_tc_eight_byte_records(k, stride, pad):
    """C = 32 with 2-bit activations: 8-byte pixel records (detection-stack first stage)."""
    c = wl.single_conv_case(seed=40 + k + stride, N=2, C=32, H=20, W=22, O=64, k=k, stride=stride, pad=pad, calibrated=True)
    acc, packed = run_tc(c)
    want = oracle.conv2d_i32(c["x"], c["w"], stride, pad)
    assert np.array_equal(acc, want)
    codes = oracle.requantize(want, c["scale"], c["bias"], True, 2, 0)
    assert np.array_equal(packed, oracle.pack_activations(codes, 2, 0))


def test_tc_chained_layers_match_oracle():
    """Three dependent layers launched back to back through the chained entry point (set-up overlapping the
    preceding kernel) give the oracle's codes, residual from the first tensor included."""
    rng = np.random.default_rng(77)
    N, C, H, W = 8, 64, 28, 28
    codes0 = wl.rand_codes(rng, (N, C, H, W), 2, wl.UNSIGNED)
    ws = [wl.rand_weights_zero_mean(rng, (C, C, 3, 3), 2, wl.SIGNED) for _ in range(3)]
    sb = [wl.calibrated_scale_bias(w, 2, 0, 2, res_scale=0.5 if i == 2 else 0.0, res_bits=2 if i == 2 else 0)
          for i, w in enumerate(ws)]
    x0 = api.bitpack_activations(dev(codes0), 1.0, 2, api.UNSIGNED, api.NCHW)
    wp = [api.pack_weights(dev(w), 2, api.SIGNED) for w in ws]
    wt = [api.tc_prepare_weights(p, C, api.SIGNED, 2) for p in wp]
    sc = [(dev(s), dev(b)) for s, b in sb]
    torch.cuda.synchronize()
    for rep in range(3):
        cur = x0
        for i in range(3):
            _, cur = api.bitserial_conv2d(cur, wp[i], C=C, stride=1, pad=1, w_sign=api.SIGNED, scale=sc[i][0], bias=sc[i][1],
                                          relu=True, out_bits=2, residual=x0 if i == 2 else None, res_scale=0.5 if i == 2 else 0.0,
                                          res_bits=2 if i == 2 else 0, res_c_total=C, wgt_tc=wt[i], chained=True)
    api.bs_check_status()
    ref = codes0
    for i in range(3):
        acc = oracle.conv2d_i32(ref, ws[i], 1, 1)
        ref = oracle.requantize(acc, sb[i][0], sb[i][1], True, 2, 0, res=codes0 if i == 2 else None, res_scale=0.5 if i == 2 else 0.0)
    assert np.array_equal(cur.cpu().numpy().view(np.uint32), oracle.pack_activations(ref, 2, 0))


def test_tc_residual_matches_oracle_and_popcount_path():
    c = wl.single_conv_case(seed=9, N=2, C=64, H=12, W=12, O=64, calibrated=True)
    rng = np.random.default_rng(4)
    res = wl.rand_codes(rng, (2, 64, 12, 12), 2, 0)
    acc, packed = run_tc(c, residual=res, res_scale=0.5)
    want = oracle.conv2d_i32(c["x"], c["w"], 1, 1)
    assert np.array_equal(acc, want)
    codes = oracle.requantize(want, c["scale"], c["bias"], True, 2, 0, res=res, res_scale=0.5)
    assert np.array_equal(packed, oracle.pack_activations(codes, 2, 0))


@pytest.mark.parametrize("kind", ["extreme_positive", "mixed_sign"])
@pytest.mark.parametrize("with_res", [False, True])
@pytest.mark.parametrize("out", [(2, 0), (2, 1), (1, 0), (1, 2)])
def test_tc_epilogue_scale_bias_corner_cases(kind, with_res, out):
    """Per-filter scales and biases at the corners of the comparison epilogue: tiny and huge positive scales with
    biases that push every threshold out of the accumulator range (integer thresholds saturate), and filters with
    zero or negative scale (the kernel must fall back to the floating-point comparison)."""
    out_bits, out_sign = out
    c = wl.single_conv_case(seed=31, N=2, C=64, H=13, W=13, O=96, calibrated=True)
    rng = np.random.default_rng(5)
    scale, bias = c["scale"].copy(), c["bias"].copy()
    O = scale.shape[0]
    scale[0::7] = 1e-6; scale[1::7] = 3e5; scale[2::7] = 1e-30
    bias[0::5] = 1e6; bias[1::5] = -1e6; bias[2::5] = 0.5; bias[3::5] = 2.5
    if kind == "mixed_sign":
        scale[3::11] *= -1.0
        scale[4::11] = 0.0
    res = wl.rand_codes(rng, (2, O, 13, 13), 2, 0) if with_res else None
    xa = api.bitpack_activations(dev(c["x"]), 1.0, 2, 0, api.NCHW)
    wp = api.pack_weights(dev(c["w"]), 2, c["w_sign"], api.NCHW)
    wt = api.tc_prepare_weights(wp, 64, c["w_sign"], 2)
    res_t = api.bitpack_activations(dev(res), 1.0, 2, 0, api.NCHW) if with_res else None
    _, packed = api.bitserial_conv2d(xa, wp, C=64, stride=1, pad=1, w_sign=c["w_sign"], scale=dev(scale), bias=dev(bias), relu=True,
                                     out_bits=out_bits, out_sign=out_sign, residual=res_t, res_scale=0.75 if with_res else 0.0,
                                     res_bits=2 if with_res else 0, res_c_total=O if with_res else 0, wgt_tc=wt)
    api.bs_check_status()
    want = oracle.conv2d_i32(c["x"], c["w"], 1, 1)
    codes = oracle.requantize(want, scale, bias, True, out_bits, out_sign, res=res, res_scale=0.75 if with_res else 0.0)
    assert np.array_equal(words(packed), oracle.pack_activations(codes, out_bits, out_sign))


@pytest.mark.parametrize("out_bits,out_sign", [(3, 0), (4, 0), (3, 1), (4, 1)])
@pytest.mark.parametrize("with_res", [False, True])
def test_tc_wide_output_codes(out_bits, out_sign, with_res):
    """3- and 4-bit outputs take the formula epilogue (no comparison form); with a 3-bit signed residual on top."""
    c = wl.single_conv_case(seed=77, N=2, C=64, H=11, W=13, O=72, calibrated=True)
    rng = np.random.default_rng(9)
    scale = (c["scale"] * (2 ** (out_bits - 2))).astype(np.float32)
    bias = (c["bias"] * (2 ** (out_bits - 2)) - (2 ** (out_bits - 1) if out_sign else 0)).astype(np.float32)
    res = wl.rand_codes(rng, (2, 72, 11, 13), 3, 1) if with_res else None
    xa = api.bitpack_activations(dev(c["x"]), 1.0, 2, 0, api.NCHW)
    wp = api.pack_weights(dev(c["w"]), 2, c["w_sign"], api.NCHW)
    wt = api.tc_prepare_weights(wp, 64, c["w_sign"], 2)
    res_t = api.bitpack_activations(dev(res), 1.0, 3, 1, api.NCHW) if with_res else None
    _, packed = api.bitserial_conv2d(xa, wp, C=64, stride=1, pad=1, w_sign=c["w_sign"], scale=dev(scale), bias=dev(bias), relu=False,
                                     out_bits=out_bits, out_sign=out_sign, residual=res_t, res_scale=0.3 if with_res else 0.0,
                                     res_bits=3 if with_res else 0, res_sign=1, res_c_total=72 if with_res else 0, wgt_tc=wt)
    api.bs_check_status()
    want = oracle.conv2d_i32(c["x"], c["w"], 1, 1)
    codes = oracle.requantize(want, scale, bias, False, out_bits, out_sign, res=res, res_scale=0.3 if with_res else 0.0)
    assert len(np.unique(codes)) >= 4
    assert np.array_equal(words(packed), oracle.pack_activations(codes, out_bits, out_sign))


@pytest.mark.parametrize("M,N,K", [(1, 8, 64), (130, 40, 128), (300, 72, 1024), (1031, 96, 64), (256, 256, 576), (1024, 1024, 2304)])
def test_tc_gemm(M, N, K):
    c = wl.gemm_case(M, N, K, seed=M + N + K)
    ap = api.bs_pack_rows(dev(c["a"]), 2, 0)
    wp = api.bs_pack_rows(dev(c["w"]), 1, 2)
    wt = api.tc_prepare_weights(wp.view(N, 1, 1, -1, 1), K, 2, 2)
    guard = Guarded()
    out, _ = api.bitserial_gemm_tc(ap, wt, N, K, 1, a_sign=0, w_sign=2, out_i32=guard.empty((M, N)))
    api.bs_check_status()
    guard.check()
    assert np.array_equal(out.cpu().numpy(), oracle.gemm_i32(c["a"], c["w"]))


@pytest.mark.parametrize("M,N,K", [(4096, 4096, 576), (4096, 4096, 4608), (4000, 4608, 3200)])
def test_tc_gemm_4096_sampled(M, N, K):
    """The largest shapes of the matrix-product sweep on the tensor-core entry point: the oracle evaluates sampled rows
    and columns; row and column sums of the whole product are checked against sums formed from the operands (a property
    that holds at any size); the requantised output is compared on the sampled rows.  K = 4608 and 3200 stage the packed
    rows in segments; 4000 x 4608 x 3200 has a last pixel tile of 32 rows and a last segment of 56 of 72 words."""
    c = wl.gemm_case(M, N, K, seed=wl.gemm_sweep_seed(M, K) if M == 4096 else 2100 + K)
    scale, bias = wl.calibrated_scale_bias(c["w"], 2, 0, 2)
    ap = api.bs_pack_rows(dev(c["a"]), 2, 0)
    wp = api.bs_pack_rows(dev(c["w"]), 1, 2)
    wt = api.tc_prepare_weights(wp.view(N, 1, 1, -1, 1), K, 2, 2)
    guard = Guarded()
    out, packed = api.bitserial_gemm_tc(ap, wt, N, K, 1, a_sign=0, w_sign=2, scale=dev(scale), bias=dev(bias), relu=True, out_bits=2,
                                        out_i32=guard.empty((M, N)), out_packed=guard.empty((M, N // 32, 2), fill=0))
    api.bs_check_status()
    guard.check()
    out = out.cpu().numpy()
    rng = np.random.default_rng(2)
    rows = np.sort(rng.choice(M, 48, replace=False))
    cols = np.sort(rng.choice(N, 48, replace=False))
    want_rows = oracle.gemm_i32(c["a"][rows], c["w"])
    assert np.array_equal(out[rows], want_rows)
    assert np.array_equal(out[:, cols], oracle.gemm_i32(c["a"], c["w"][cols]))
    wsum = c["w"].astype(np.int64).sum(axis=0)
    assert np.array_equal(out.astype(np.int64).sum(axis=1), c["a"].astype(np.int64) @ wsum)
    asum = c["a"].astype(np.int64).sum(axis=0)
    assert np.array_equal(out.astype(np.int64).sum(axis=0), c["w"].astype(np.int64) @ asum)
    codes = oracle.requantize(want_rows, scale, bias, True, 2, 0, channel_axis=1)
    assert len(np.unique(codes)) == 4
    assert np.array_equal(words(packed)[rows], oracle.pack_rows(codes, 2, 0))


def test_tc_unsupported_shape_is_refused():
    assert api.tc_supported(1, 32, 8, 8, 32, 3, 1, 1, 2, 0, 2, 1)           # 8-byte records on 16-byte rows are fine
    assert not api.tc_supported(1, 32, 8, 7, 32, 3, 1, 1, 2, 0, 2, 1)       # ... but not on odd-width images
    assert not api.tc_supported(1, 32, 8, 8, 32, 3, 1, 1, 1, 0, 2, 1)       # 4-byte records cannot be fetched in bulk
    assert not api.tc_supported(1, 40, 8, 8, 32, 3, 1, 1, 4, 0, 2, 1)       # C not a multiple of 32
    assert api.tc_supported(1, 64, 8, 8, 32, 3, 1, 1, 2, 0, 2, 1)
