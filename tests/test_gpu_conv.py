"""GPU parity: bitserial_conv2d against the oracle's direct integer convolution (bit-exact int32) and
its requantisation epilogue (tolerance: at most 1e-4 of the codes may differ, by at most one level;
zero differences are expected because both sides run the same binary32 operations)."""
import numpy as np
import pytest
import torch

import oracle
from paper_2207_08820_b200 import api, workloads as wl
from gpu_util import dev, gpu_conv, words

pytestmark = pytest.mark.gpu

REQUANT_MAX_FRACTION = 1e-4


def assert_codes_close(got_codes, want_codes):
    diff = np.abs(got_codes.astype(np.int32) - want_codes.astype(np.int32))
    assert diff.max(initial=0) <= 1
    assert (diff != 0).mean() <= REQUANT_MAX_FRACTION


def packed_to_codes(packed_words, C, bits, sign):
    return oracle.unpack_activations(packed_words, C, bits, sign)


def test_single_layer_seed0_literal_and_calibrated():
    """3x3, stride 1, pad 1, 1x64x56x56, 64 filters, 2-bit/2-bit, seed 0: accumulators bit-exact; requantised
    output with the literal scale/bias draw and with the calibrated draw that exercises every level."""
    for calibrated in (False, True):
        c = wl.single_conv_case(seed=0, calibrated=calibrated)
        acc, packed = gpu_conv(c)
        want_acc = oracle.conv2d_i32(c["x"], c["w"], 1, 1)
        assert np.array_equal(acc, want_acc)
        want_codes = oracle.requantize(want_acc, c["scale"], c["bias"], True, 2, 0)
        if calibrated:
            assert len(np.unique(want_codes)) == 4
        assert_codes_close(packed_to_codes(packed, 64, 2, 0), want_codes)
        assert np.array_equal(packed, oracle.pack_activations(want_codes, 2, 0))


@pytest.mark.parametrize("k,stride,pad", [(1, 1, 0), (1, 2, 0), (3, 1, 1), (3, 2, 1), (3, 1, 0), (3, 2, 0), (5, 1, 2), (7, 2, 3)])
@pytest.mark.parametrize("hw", [(5, 5), (7, 9), (9, 6), (8, 8)])
def test_conv_geometry(k, stride, pad, hw):
    H, W = hw
    if H + 2 * pad < k or W + 2 * pad < k:
        pytest.skip("kernel larger than padded image")
    c = wl.single_conv_case(seed=k * 100 + stride * 10 + pad + H, N=3, C=40, H=H, W=W, O=24, k=k, stride=stride, pad=pad,
                            calibrated=True)
    acc, packed = gpu_conv(c)
    want = oracle.conv2d_i32(c["x"], c["w"], stride, pad)
    assert np.array_equal(acc, want)
    codes = oracle.requantize(want, c["scale"], c["bias"], True, 2, 0)
    assert np.array_equal(packed, oracle.pack_activations(codes, 2, 0))


@pytest.mark.parametrize("wb", [1, 2, 3, 4])
@pytest.mark.parametrize("ab", [1, 2, 3, 4])
@pytest.mark.parametrize("signs", [(0, None), (1, None), (0, 0)])
def test_conv_all_bitwidths(wb, ab, signs):
    a_sign, w_sign = signs
    if a_sign == 1 and ab == 1:
        pytest.skip("1-bit two's complement activations are not offered")
    c = wl.single_conv_case(seed=wb * 10 + ab, N=2, C=96, H=10, W=9, O=40, a_bits=ab, w_bits=wb, a_sign=a_sign,
                            w_sign=w_sign, out_bits=ab, calibrated=True)
    acc, packed = gpu_conv(c, i32_layout=api.NHWC)
    want = oracle.conv2d_i32(c["x"], c["w"], 1, 1)
    assert np.array_equal(acc, want.transpose(0, 2, 3, 1))
    codes = oracle.requantize(want, c["scale"], c["bias"], True, ab, 0)
    assert np.array_equal(packed, oracle.pack_activations(codes, ab, 0))


def test_conv_bipolar_activations_no_padding():
    for wsg, wb in ((2, 1), (1, 2), (0, 2)):
        c = wl.single_conv_case(seed=77 + wb, N=2, C=70, H=8, W=8, O=33, k=3, pad=0, a_bits=1, a_sign=2, w_bits=wb, w_sign=wsg)
        acc, _ = gpu_conv(c, want_packed=False)
        assert np.array_equal(acc, oracle.conv2d_i32(c["x"], c["w"], 1, 0))


def test_conv_border_closed_form():
    """Top-code activations and all +1 (bipolar) weights: acc = amax * C * (taps inside the image)."""
    C, H, W, O = 64, 12, 17, 32
    c = wl.single_conv_case(seed=1, N=1, C=C, H=H, W=W, O=O, w_bits=1)
    c["x"][:] = 3
    c["w"][:] = 1
    acc, _ = gpu_conv(c, want_packed=False)
    ty = np.array([2 if y in (0, H - 1) else 3 for y in range(H)])
    tx = np.array([2 if x in (0, W - 1) else 3 for x in range(W)])
    want = 3 * C * np.outer(ty, tx)
    for o in range(O):
        assert np.array_equal(acc[0, o], want)


@pytest.mark.parametrize("C,O", [(32, 32), (64, 128), (128, 64), (256, 96), (512, 64), (33, 31)])
def test_conv_channel_counts(C, O):
    c = wl.single_conv_case(seed=C + O, N=2, C=C, H=14, W=14, O=O, calibrated=True)
    acc, packed = gpu_conv(c)
    want = oracle.conv2d_i32(c["x"], c["w"], 1, 1)
    assert np.array_equal(acc, want)
    codes = oracle.requantize(want, c["scale"], c["bias"], True, 2, 0)
    assert np.array_equal(packed, oracle.pack_activations(codes, 2, 0))


def test_conv_residual_and_concat():
    """Residual operand in the epilogue and writing at a channel offset of a wider output tensor."""
    c = wl.single_conv_case(seed=9, N=2, C=64, H=12, W=12, O=64, calibrated=True)
    rng = np.random.default_rng(4)
    res = wl.rand_codes(rng, (2, 96, 12, 12), 2, 0)            # residual taken from channels 32..95
    total = 160
    out = torch.full((2, 12, 12, total // 32, 2), -1, dtype=torch.int32, device="cuda")
    acc, packed = gpu_conv(c, residual=(res, 2, 0), res_scale=0.5, res_c_offset=32, out_c_offset=64, out_c_total=total,
                           out_packed=out)
    want = oracle.conv2d_i32(c["x"], c["w"], 1, 1)
    assert np.array_equal(acc, want)
    codes = oracle.requantize(want, c["scale"], c["bias"], True, 2, 0, res=res[:, 32:96], res_scale=0.5)
    want_words = oracle.pack_activations(codes, 2, 0)
    assert np.array_equal(packed[:, :, :, 2:4, :], want_words)
    assert np.all(packed[:, :, :, :2, :] == 0xFFFFFFFF) and np.all(packed[:, :, :, 4:, :] == 0xFFFFFFFF)


def test_conv_1x1_equals_gemm_bytes():
    """A 1x1 convolution and a matrix product over the same packed bytes give the same accumulators."""
    c = wl.single_conv_case(seed=12, N=2, C=100, H=6, W=7, O=48, k=1, pad=0)
    acc, _ = gpu_conv(c, want_packed=False, i32_layout=api.NHWC)
    xa = api.bitpack_activations(dev(c["x"]), 1.0, 2, 0, api.NCHW)
    wp = api.pack_weights(dev(c["w"]), 2, 1, api.NCHW)
    out, _ = api.bitserial_gemm(xa.view(2 * 6 * 7, 4, 2), wp.view(48, 4, 2), 100, a_sign=0, w_sign=1)
    assert np.array_equal(out.cpu().numpy().reshape(2, 6, 7, 48), acc)
    assert np.array_equal(acc, oracle.conv2d_i32(c["x"], c["w"], 1, 0).transpose(0, 2, 3, 1))


@pytest.mark.parametrize("wb,ab", wl.BITWIDTH_SWEEP)
def test_bitwidth_sweep_full_size_sampled(wb, ab):
    """3x3 conv, N=32, C=O=256, 28x28 at full size: the oracle evaluates three sampled images."""
    c = wl.bitwidth_sweep_case(wb, ab)
    acc, packed = gpu_conv(c)
    for n in (0, 13, 31):
        want = oracle.conv2d_i32(c["x"][n:n + 1], c["w"], 1, 1)
        assert np.array_equal(acc[n:n + 1], want)
        codes = oracle.requantize(want, c["scale"], c["bias"], True, ab, 0)
        assert np.array_equal(packed[n:n + 1], oracle.pack_activations(codes, ab, 0))
