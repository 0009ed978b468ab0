"""GPU parity: quantise + bitplane packing kernels against the oracle, bit for bit."""
import numpy as np
import pytest
import torch

import oracle
from paper_2207_08820_b200 import api, workloads as wl
from gpu_util import dev, words

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("bits,sign", [(1, 0), (2, 0), (3, 0), (4, 0), (2, 1), (3, 1), (4, 1), (1, 2)])
@pytest.mark.parametrize("shape", [(1, 64, 56, 56), (2, 45, 7, 9), (3, 32, 5, 5), (1, 200, 3, 130), (2, 96, 20, 20)])
def test_bitpack_fp32_nchw_matches_oracle(bits, sign, shape):
    rng = np.random.default_rng(bits * 100 + sign * 10 + shape[1])
    s = 0.37
    lo, hi = wl.code_range(bits, sign)
    x = rng.uniform((lo - 1.5) * s, (hi + 1.5) * s, size=shape).astype(np.float32)
    # plant exact ties: x/s = k + 0.5 in binary32
    ties = (np.arange(x.size // 7, dtype=np.float32) % (hi - lo + 2) + lo - 0.5)
    x.reshape(-1)[: ties.size] = ties * np.float32(s)
    want = oracle.pack_activations(oracle.quantize(x, s, bits, sign), bits, sign)
    got = words(api.bitpack_activations(dev(x), s, bits, sign, api.NCHW))
    assert np.array_equal(got, want)


@pytest.mark.parametrize("bits,sign", [(1, 0), (2, 0), (2, 1), (1, 2), (3, 0)])
@pytest.mark.parametrize("s", [0.37, 1.0, 2.5e-3, 1e-38])
def test_bitpack_special_values(bits, sign, s):
    """NaN, infinities, signed zeros, denormals and the neighbours of every rounding tie: the sign-bit form of the
    quantiser must take the decision of the Section IV formula on all of them."""
    lo, hi = wl.code_range(bits, sign)
    s32 = np.float32(s)
    ties = (np.arange(lo - 1, hi + 2, dtype=np.float32) + np.float32(0.5)) * s32
    near = np.concatenate([ties, np.nextafter(ties, np.float32(np.inf)), np.nextafter(ties, np.float32(-np.inf)),
                           np.arange(lo - 1, hi + 2, dtype=np.float32) * s32])
    special = np.array([np.nan, np.inf, -np.inf, 0.0, -0.0, 1e-45, -1e-45, 1e-39, -1e-39, 3e38, -3e38, 1.0, -1.0], dtype=np.float32)
    vals = np.concatenate([near, special]).astype(np.float32)
    rng = np.random.default_rng(3)
    x = rng.choice(vals, size=(2, 64, 6, 17)).astype(np.float32)
    with np.errstate(all="ignore"):
        want = oracle.pack_activations(oracle.quantize(x, s, bits, sign), bits, sign)
    got = words(api.bitpack_activations(dev(x), s, bits, sign, api.NCHW))
    assert np.array_equal(got, want)
    got = words(api.bitpack_activations(dev(np.ascontiguousarray(x.transpose(0, 2, 3, 1))), s, bits, sign, api.NHWC))
    assert np.array_equal(got, want)


@pytest.mark.parametrize("bits,sign", [(2, 0), (3, 1), (1, 2)])
@pytest.mark.parametrize("shape", [(2, 64, 9, 11), (1, 70, 6, 50)])
def test_bitpack_nhwc_and_int8_inputs(bits, sign, shape):
    rng = np.random.default_rng(bits + sign)
    N, C, H, W = shape
    s = 0.5
    lo, hi = wl.code_range(bits, sign)
    x = rng.uniform((lo - 1) * s, (hi + 1) * s, size=shape).astype(np.float32)
    codes = oracle.quantize(x, s, bits, sign)
    want = oracle.pack_activations(codes, bits, sign)
    got = words(api.bitpack_activations(dev(x.transpose(0, 2, 3, 1)), s, bits, sign, api.NHWC))
    assert np.array_equal(got, want)
    got = words(api.bitpack_activations(dev(codes), 1.0, bits, sign, api.NCHW))
    assert np.array_equal(got, want)
    got = words(api.bitpack_activations(dev(codes.transpose(0, 2, 3, 1)), 1.0, bits, sign, api.NHWC))
    assert np.array_equal(got, want)


@pytest.mark.parametrize("bits,sign", [(1, 0), (2, 0), (3, 0), (4, 0), (1, 1), (2, 1), (3, 1), (4, 1), (1, 2)])
@pytest.mark.parametrize("shape", [(2, 64, 8, 12), (1, 96, 7, 20), (3, 32, 6, 6), (1, 45, 4, 33), (2, 128, 13, 20), (1, 32, 1, 4)])
def test_bitpack_vector_paths_all_layouts(bits, sign, shape):
    """Shapes that reach the kernels with one (pixels, channel word) unit per warp: H*W a multiple of 4 (int8 NCHW reads
    four pixels per word), C a multiple of 32 (int8 NHWC reads 32 channels per lane), ragged last tiles of 32 and of 128
    pixels, a ragged last channel word; fp32 and int8 inputs in both layouts against the oracle, bit for bit."""
    rng = np.random.default_rng(bits * 10 + sign + shape[1])
    s = 0.61
    lo, hi = wl.code_range(bits, sign)
    x = rng.uniform((lo - 1.2) * s, (hi + 1.2) * s, size=shape).astype(np.float32)
    codes = oracle.quantize(x, s, bits, sign)
    want = oracle.pack_activations(codes, bits, sign)
    assert np.array_equal(words(api.bitpack_activations(dev(x), s, bits, sign, api.NCHW)), want)
    assert np.array_equal(words(api.bitpack_activations(dev(x.transpose(0, 2, 3, 1)), s, bits, sign, api.NHWC)), want)
    assert np.array_equal(words(api.bitpack_activations(dev(codes), 1.0, bits, sign, api.NCHW)), want)
    assert np.array_equal(words(api.bitpack_activations(dev(codes.transpose(0, 2, 3, 1)), 1.0, bits, sign, api.NHWC)), want)


@pytest.mark.parametrize("bits,sign", [(1, 0), (2, 0), (4, 1), (1, 2)])
def test_unpack_is_inverse(bits, sign):
    rng = np.random.default_rng(3)
    codes = wl.rand_codes(rng, (2, 77, 6, 5), bits, sign)
    packed = api.bitpack_activations(dev(codes), 1.0, bits, sign, api.NCHW)
    assert np.array_equal(api.bitunpack_activations(packed, 77, bits, sign, api.NCHW).cpu().numpy(), codes)
    assert np.array_equal(api.bitunpack_activations(packed, 77, bits, sign, api.NHWC).cpu().numpy(),
                          codes.transpose(0, 2, 3, 1))


@pytest.mark.parametrize("bits,sign", [(1, 2), (1, 0), (2, 1), (3, 1), (4, 1), (2, 0)])
def test_pack_weights_and_rows(bits, sign):
    rng = np.random.default_rng(bits * 3 + sign)
    w = wl.rand_codes(rng, (37, 70, 3, 3), bits, sign)
    want = oracle.pack_weights(w, bits, sign)
    assert np.array_equal(words(api.pack_weights(dev(w), bits, sign, api.NCHW)), want)
    assert np.array_equal(words(api.pack_weights(dev(w.transpose(0, 2, 3, 1)), bits, sign, api.NHWC)), want)
    rows = wl.rand_codes(rng, (53, 577), bits, sign)
    assert np.array_equal(words(api.bs_pack_rows(dev(rows), bits, sign)), oracle.pack_rows(rows, bits, sign))


def test_bitpack_full_size_first_layer_sampled():
    """Full-size first-layer tensor of the residual stack (64 x 64 x 56 x 56): the oracle packs three
    sampled images; the rest is checked through the unpack round trip against the oracle quantiser."""
    net = wl.resnet18_body(64)
    x = wl.network_input(net, seed=3000)
    packed = api.bitpack_activations(dev(x), 0.25, 2, 0, api.NCHW)
    got = words(packed)
    for n in (0, 17, 63):
        want = oracle.pack_activations(oracle.quantize(x[n:n + 1], 0.25, 2, 0), 2, 0)
        assert np.array_equal(got[n:n + 1], want)
    codes = api.bitunpack_activations(packed, 64, 2, 0, api.NCHW).cpu().numpy()
    assert np.array_equal(codes, oracle.quantize(x, 0.25, 2, 0))
