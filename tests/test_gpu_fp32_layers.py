"""GPU parity for the layers kept in floating point (stem convolution, max pool, average pool of codes, fully connected)
and for the whole mixed-precision classifier.  The kernels follow the oracle's operation order, so float32 results are
compared for equality, bit for bit; the whole network is compared tensor by tensor (codes: at most 1e-4 of elements off
by one level, zero expected; logits: equal)."""
import numpy as np
import pytest
import torch

import oracle
from oracle import network as onet
from paper_2207_08820_b200 import api, workloads as wl
from paper_2207_08820_b200.net import BitserialFullNet
from gpu_util import dev

pytestmark = pytest.mark.gpu


def same_bits(a: np.ndarray, b: np.ndarray) -> bool:
    return a.shape == b.shape and np.array_equal(a.view(np.uint32), b.view(np.uint32))


@pytest.mark.parametrize("C,O,k,stride,pad,hw", [(3, 64, 7, 2, 3, (37, 45)), (3, 64, 7, 2, 3, (224, 224)), (3, 40, 7, 2, 3, (20, 21)),
                                                 (5, 70, 3, 1, 1, (13, 34)), (4, 64, 3, 2, 1, (17, 9)), (8, 16, 1, 1, 0, (6, 50)),
                                                 (3, 8, 5, 1, 2, (11, 12)), (2, 3, 4, 3, 0, (15, 16))])
@pytest.mark.parametrize("relu", [False, True])
def test_conv2d_f32_bit_exact(C, O, k, stride, pad, hw, relu):
    rng = np.random.default_rng(C * 100 + O + k)
    H, W = hw
    N = 2 if H < 100 else 1
    x = rng.normal(0, 1, (N, C, H, W)).astype(np.float32)
    w = (rng.normal(0, 1, (O, C, k, k)) / np.sqrt(C * k * k)).astype(np.float32)
    b = rng.normal(0, 0.5, O).astype(np.float32)
    got = api.conv2d_f32(dev(x), dev(w), dev(b), stride, pad, relu).cpu().numpy()
    api.bs_check_status()
    assert same_bits(got, oracle.conv2d_f32(x, w, b, stride, pad, relu))
    got_nb = api.conv2d_f32(dev(x), dev(w), None, stride, pad, relu).cpu().numpy()
    assert same_bits(got_nb, oracle.conv2d_f32(x, w, None, stride, pad, relu))


def test_conv2d_f32_summation_order_witness():
    """2^24 + 1 rounds back to 2^24: channel order (2^24, 1, -2^24) must give 0 and (2^24, -2^24, 1) must give 1, on the
    tiled kernel (1x1) and on the generic one (2x1 kernel)."""
    big = np.float32(16777216.0)
    for vals, want in (((big, 1.0, -big), 0.0), ((big, -big, 1.0), 1.0)):
        x = np.array(vals, dtype=np.float32).reshape(1, 3, 1, 1).repeat(8, axis=3)
        w = np.ones((4, 3, 1, 1), dtype=np.float32)
        got = api.conv2d_f32(dev(x), dev(w)).cpu().numpy()
        assert np.all(got == want)
    x = np.array([big, -big, 1.0, 0.0], dtype=np.float32).reshape(1, 2, 2, 1)
    got = api.conv2d_f32(dev(x), dev(np.ones((1, 2, 2, 1), dtype=np.float32))).cpu().numpy()
    assert got.reshape(-1)[0] == 1.0


@pytest.mark.parametrize("k,stride,pad", [(3, 2, 1), (2, 2, 0), (3, 1, 1)])
def test_maxpool_bit_exact(k, stride, pad):
    rng = np.random.default_rng(k)
    x = rng.normal(-1, 1, (3, 6, 29, 18)).astype(np.float32)
    got = api.maxpool2d_f32(dev(x), k, stride, pad).cpu().numpy()
    assert same_bits(got, oracle.maxpool2d_f32(x, k, stride, pad))
    # a row width that is a multiple of 8 takes the vectorised kernel when the window is 3x3, stride 2, pad 1
    x8 = rng.normal(-1, 1, (2, 5, 13, 24)).astype(np.float32)
    got8 = api.maxpool2d_f32(dev(x8), k, stride, pad).cpu().numpy()
    assert same_bits(got8, oracle.maxpool2d_f32(x8, k, stride, pad))


@pytest.mark.parametrize("bits,sign,C", [(2, 0, 512), (3, 1, 70), (1, 2, 33), (4, 0, 64)])
def test_avgpool_codes_bit_exact(bits, sign, C):
    rng = np.random.default_rng(bits + C)
    codes = wl.rand_codes(rng, (5, C, 7, 7), bits, sign)
    packed = api.bitpack_activations(dev(codes), 1.0, bits, sign, api.NCHW)
    inv = float(np.float32(np.float32(0.25) / np.float32(49)))
    got = api.avgpool_codes_f32(packed, C, sign, inv).cpu().numpy()
    assert same_bits(got, oracle.avgpool_codes(codes, inv))


@pytest.mark.parametrize("N,K,J", [(64, 512, 1000), (3, 70, 5), (9, 64, 33), (1, 1, 1)])
def test_fc_bit_exact(N, K, J):
    rng = np.random.default_rng(N + K + J)
    x = rng.normal(0, 1, (N, K)).astype(np.float32)
    w = (rng.normal(0, 1, (J, K)) / np.sqrt(K)).astype(np.float32)
    b = rng.normal(0, 1, J).astype(np.float32)
    got = api.fc_f32(dev(x), dev(w), dev(b)).cpu().numpy()
    assert same_bits(got, oracle.fc_f32(x, w, b))


@pytest.mark.parametrize("engine", ["tc", "popc"])
def test_full_classifier_every_tensor(engine):
    """Whole mixed-precision network at 64 x 64 input, batch 3, free-running on both sides from the same images."""
    net = wl.resnet18_full(batch=3, hw=64)
    params = wl.full_network_params(net, 8100)
    images = wl.full_network_input(net, 8100)
    runner = BitserialFullNet(net, params, batch=3, engine=engine)
    logits = runner.forward(dev(images)).cpu().numpy()
    api.bs_check_status()
    want = onet.run_full(net, params, images)
    assert same_bits(runner.stem_conv.cpu().numpy(), want["stem_conv"])
    assert same_bits(runner.stem_pool.cpu().numpy(), want["stem_pool"])
    levels = set()
    for name in net.body.tensor_shapes():
        got = runner.body.unpacked(name).cpu().numpy()
        diff = np.abs(got.astype(np.int32) - want[name].astype(np.int32))
        assert diff.max() <= 1 and (diff != 0).mean() <= 1e-4, name
        levels |= set(np.unique(want[name]).tolist())
    assert levels == {0, 1, 2, 3}
    assert same_bits(runner.pooled.cpu().numpy(), want["pooled"])
    assert same_bits(logits, want["logits"])
    assert np.unique(np.argmax(logits, axis=1)).size >= 1 and np.std(logits) > 0.05


def test_full_classifier_full_size_sampled():
    """224 x 224, batch 64 (the size the benchmark times): the oracle runs two sampled images."""
    net = wl.resnet18_full(batch=64)
    params = wl.full_network_params(net, 8200)
    images = wl.full_network_input(net, 8200)
    runner = BitserialFullNet(net, params, batch=64, engine="tc")
    logits = runner.forward(dev(images)).cpu().numpy()
    api.bs_check_status()
    idx = [0, 63]
    want = onet.run_full(net, params, images[idx])
    assert same_bits(runner.stem_pool.cpu().numpy()[idx], want["stem_pool"])
    out = net.body.out_name
    assert np.array_equal(runner.body.unpacked(out).cpu().numpy()[idx], want[out])
    assert same_bits(logits[idx], want["logits"])
