"""GPU parity: bitserial_gemm against the oracle's plain integer matrix product (bit-exact int32)."""
import numpy as np
import pytest

import oracle
from paper_2207_08820_b200 import api, workloads as wl
from gpu_util import Guarded, dev, words

pytestmark = pytest.mark.gpu


def run_gemm(c, **kw):
    ap = api.bs_pack_rows(dev(c["a"]), c["a_bits"], c["a_sign"])
    wp = api.bs_pack_rows(dev(c["w"]), c["w_bits"], c["w_sign"])
    guard = Guarded()
    M, N = c["a"].shape[0], c["w"].shape[0]
    out_i32 = guard.empty((M, N))
    out_packed = guard.empty((M, (N + 31) // 32, kw["out_bits"]), fill=0) if kw.get("out_bits", 0) else None
    out, packed = api.bitserial_gemm(ap, wp, c["K"], a_sign=c["a_sign"], w_sign=c["w_sign"], out_i32=out_i32,
                                     out_packed=out_packed, **kw)
    api.bs_check_status()
    guard.check()
    return out, packed


@pytest.mark.parametrize("ab,asg", [(1, 0), (2, 0), (3, 0), (4, 0), (2, 1), (3, 1), (1, 2)])
@pytest.mark.parametrize("wb,wsg", [(1, 2), (1, 0), (2, 1), (3, 1), (4, 1), (2, 0)])
def test_gemm_all_bitwidths_and_signs(ab, asg, wb, wsg):
    c = wl.gemm_case(67, 45, 203, seed=ab * 1000 + asg * 100 + wb * 10 + wsg, a_bits=ab, a_sign=asg, w_bits=wb, w_sign=wsg)
    out, _ = run_gemm(c)
    assert np.array_equal(out.cpu().numpy(), oracle.gemm_i32(c["a"], c["w"]))


@pytest.mark.parametrize("M,N,K", [(1, 1, 1), (5, 3, 31), (8, 64, 32), (300, 70, 33), (257, 129, 1000), (1031, 96, 64),
                                   (256, 256, 576), (64, 520, 4608)])
def test_gemm_ragged_shapes_bipolar_weights(M, N, K):
    c = wl.gemm_case(M, N, K, seed=M + N + K)
    out, _ = run_gemm(c)
    assert np.array_equal(out.cpu().numpy(), oracle.gemm_i32(c["a"], c["w"]))


def test_gemm_requantised_output():
    c = wl.gemm_case(150, 96, 320, seed=5, a_bits=2, a_sign=0, w_bits=2, w_sign=1)
    scale, bias = wl.calibrated_scale_bias(c["w"], 2, 0, 3)
    out, packed = run_gemm(c, scale=dev(scale), bias=dev(bias), relu=True, out_bits=3, out_sign=0)
    acc = oracle.gemm_i32(c["a"], c["w"])
    assert np.array_equal(out.cpu().numpy(), acc)
    codes = oracle.requantize(acc, scale, bias, True, 3, 0, channel_axis=1)
    assert len(np.unique(codes)) == 8
    assert np.array_equal(words(packed), oracle.pack_rows(codes, 3, 0))


@pytest.mark.parametrize("M,K", [(m, k) for m in wl.GEMM_SWEEP_MN for k in wl.GEMM_SWEEP_K])
def test_gemm_sweep_full_size(M, K):
    """The nine sweep shapes (1-bit bipolar weights, 2-bit unsigned activations).  Small shapes are compared in
    full; for the large ones the oracle evaluates sampled rows and columns, and row/column sums of the
    whole product are checked against sums computed from the operands (a property that holds at any size)."""
    c = wl.gemm_case(M, M, K, seed=wl.gemm_sweep_seed(M, K))
    out = run_gemm(c)[0].cpu().numpy()
    if M <= 1024:
        assert np.array_equal(out, oracle.gemm_i32(c["a"], c["w"]))
        return
    rng = np.random.default_rng(1)
    rows = np.sort(rng.choice(M, 48, replace=False))
    cols = np.sort(rng.choice(M, 48, replace=False))
    assert np.array_equal(out[rows], oracle.gemm_i32(c["a"][rows], c["w"]))
    assert np.array_equal(out[:, cols], oracle.gemm_i32(c["a"], c["w"][cols]))
    wsum = c["w"].astype(np.int64).sum(axis=0)           # sum_n out[m][n] = a[m] . sum_n w[n]
    assert np.array_equal(out.astype(np.int64).sum(axis=1), c["a"].astype(np.int64) @ wsum)
    asum = c["a"].astype(np.int64).sum(axis=0)
    assert np.array_equal(out.astype(np.int64).sum(axis=0), c["w"].astype(np.int64) @ asum)
