"""GPU parity for the reduction split (`*_ws` entry points): bit-identical to the oracle and to the unsplit kernel,
workspace left zero, repeated calls on one workspace."""
import numpy as np
import pytest
import torch

import oracle
from paper_2207_08820_b200 import api, workloads as wl
from gpu_util import dev, words

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("M,N,K", [(256, 256, 4608), (256, 256, 576), (64, 96, 2304), (130, 40, 1000)])
@pytest.mark.parametrize("wb,wsg", [(1, 2), (2, 1)])
def test_gemm_split_matches_oracle_and_leaves_workspace_zero(M, N, K, wb, wsg):
    c = wl.gemm_case(M, N, K, seed=M + K + wb, w_bits=wb, w_sign=wsg)
    ap = api.bs_pack_rows(dev(c["a"]), 2, 0)
    wp = api.bs_pack_rows(dev(c["w"]), wb, wsg)
    ws = api.gemm_workspace(M, N, K, 2, 0, wb, wsg)
    want = oracle.gemm_i32(c["a"], c["w"])
    if ws is None:
        pytest.skip("planner does not split this shape")
    scale, bias = wl.calibrated_scale_bias(c["w"], 2, 0, 2)
    codes = oracle.requantize(want, scale, bias, True, 2, 0, channel_axis=1)
    for _ in range(3):                                   # the workspace is reused without clearing
        out, packed = api.bitserial_gemm(ap, wp, K, a_sign=0, w_sign=wsg, scale=dev(scale), bias=dev(bias), relu=True,
                                         out_bits=2, workspace=ws)
        api.bs_check_status()
        assert np.array_equal(out.cpu().numpy(), want)
        assert np.array_equal(words(packed), oracle.pack_rows(codes, 2, 0))
        assert int(ws.abs().max()) == 0
    plain, _ = api.bitserial_gemm(ap, wp, K, a_sign=0, w_sign=wsg)
    assert torch.equal(plain, out)


def test_conv_split_deep_reduction():
    """7 x 7 layer with 512 channels at batch 4: few tiles, 144 reduction words."""
    c = wl.single_conv_case(seed=21, N=4, C=512, H=7, W=7, O=512, calibrated=True)
    ws = api.conv_workspace(4, 512, 7, 7, 512, 3, 1, 1, 2, 0, 2, 1)
    assert ws is not None
    x, w = dev(c["x"]), dev(c["w"])
    xa = api.bitpack_activations(x, 1.0, 2, 0, api.NCHW)
    wp = api.pack_weights(w, 2, 1, api.NCHW)
    want = oracle.conv2d_i32(c["x"], c["w"], 1, 1)
    codes = oracle.requantize(want, c["scale"], c["bias"], True, 2, 0)
    for _ in range(2):
        acc, packed = api.bitserial_conv2d(xa, wp, C=512, stride=1, pad=1, w_sign=1, scale=dev(c["scale"]), bias=dev(c["bias"]),
                                           relu=True, out_bits=2, want_i32=True, workspace=ws)
        api.bs_check_status()
        assert np.array_equal(acc.cpu().numpy(), want)
        assert np.array_equal(words(packed), oracle.pack_activations(codes, 2, 0))
        assert int(ws.abs().max()) == 0


def test_too_small_workspace_falls_back():
    c = wl.gemm_case(256, 256, 4608, seed=3)
    ap = api.bs_pack_rows(dev(c["a"]), 2, 0)
    wp = api.bs_pack_rows(dev(c["w"]), 1, 2)
    tiny = torch.zeros(4, dtype=torch.int32, device="cuda")
    out, _ = api.bitserial_gemm(ap, wp, 4608, a_sign=0, w_sign=2, workspace=tiny)
    api.bs_check_status()
    assert np.array_equal(out.cpu().numpy(), oracle.gemm_i32(c["a"], c["w"]))
