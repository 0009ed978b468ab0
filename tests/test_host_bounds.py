"""Host logic (no GPU): the comparison forms the kernels evaluate, checked against the oracle's formulas.

`bs_quantiser_bounds` and `bs_requant_bounds` return the bounds that the pack kernels and the tensor-core epilogue
compare against.  A bound is right when the oracle's own quantiser / epilogue changes its code exactly there: at the
bound the code has reached the level, one float below it has not."""
import ctypes

import numpy as np
import pytest

import oracle
from paper_2207_08820_b200 import workloads as wl
from paper_2207_08820_b200._lib import lib

F32 = np.float32


def _below(b):
    return np.nextafter(F32(b), F32(-np.inf))


@pytest.mark.parametrize("bits,sign", [(1, 0), (2, 0), (3, 0), (4, 0), (1, 1), (2, 1), (3, 1), (4, 1), (1, 2)])
@pytest.mark.parametrize("s", [0.37, 1.0, 0.25, 2.5e-3, 1e-38, 7.3e5])
def test_quantiser_bounds_are_where_the_oracle_changes_code(bits, sign, s):
    L = lib()
    n = 1 if sign == 2 else (1 << bits) - 1
    buf = (ctypes.c_float * 15)()
    assert L.bs_quantiser_bounds(ctypes.c_float(s), bits, sign, buf) == 0
    bounds = np.array(buf[:n], dtype=F32)
    assert np.all(np.isfinite(bounds)) and np.all(np.diff(bounds) > 0)
    qmin, _ = wl.code_range(bits, sign)
    at = oracle.quantize(bounds, s, bits, sign).astype(int)
    under = oracle.quantize(_below(bounds), s, bits, sign).astype(int)
    if sign == 2:
        assert at.tolist() == [1] and under.tolist() == [-1] and bounds[0] == 0.0
    else:
        assert at.tolist() == [qmin + k + 1 for k in range(n)]
        assert under.tolist() == [qmin + k for k in range(n)]
    # the count of bounds reached is the code, on random inputs and on the rounding ties
    rng = np.random.default_rng(bits * 7 + sign)
    x = np.concatenate([rng.uniform(-12 * s, 20 * s, 4000), (np.arange(-10, 18) + 0.5) * F32(s)]).astype(F32)
    count = (x[:, None] >= bounds[None, :]).sum(axis=1)
    want = oracle.quantize(x, s, bits, sign).astype(int)
    got = np.where(count > 0, 1, -1) if sign == 2 else qmin + count
    assert np.array_equal(got, want)


def test_quantiser_bounds_reject_bad_arguments():
    L = lib()
    buf = (ctypes.c_float * 15)()
    assert L.bs_quantiser_bounds(ctypes.c_float(0.0), 2, 0, buf) == 1
    assert L.bs_quantiser_bounds(ctypes.c_float(1.0), 5, 0, buf) == 1
    assert L.bs_quantiser_bounds(ctypes.c_float(1.0), 2, 2, buf) == 1        # bipolar needs one bit
    assert L.bs_quantiser_bounds(ctypes.c_float(1.0), 2, 0, None) == 1


@pytest.mark.parametrize("out_bits,out_sign", [(1, 0), (2, 0), (1, 1), (2, 1), (1, 2)])
@pytest.mark.parametrize("relu", [0, 1])
@pytest.mark.parametrize("res", [None, (2, 0, 0.5), (2, 1, 0.75), (1, 2, 1.5), (3, 0, 0.3)])
def test_requant_bounds_are_where_the_oracle_epilogue_changes_code(out_bits, out_sign, relu, res):
    """t = fmaf(acc, scale, bias) is produced exactly with acc = 0, scale = 1, bias = t."""
    L = lib()
    buf = (ctypes.c_float * 48)()
    has_res = res is not None
    res_bits, res_sign, res_scale = res if has_res else (0, 0, 0.0)
    assert L.bs_requant_bounds(int(has_res), ctypes.c_float(res_scale), res_bits, res_sign, relu, out_bits, out_sign, buf) == 0
    npat = (1 << res_bits) if has_res else 1
    qmin, qmax = wl.code_range(out_bits, out_sign)
    nlev = 2 if out_sign == 2 else (1 << out_bits)
    for r in range(npat):
        if has_res:
            v = r - (1 << res_bits) if (res_sign == 1 and r >> (res_bits - 1)) else r
            res_code = (1 if r else -1) if res_sign == 2 else v
        bounds = np.array(buf[3 * r:3 * r + 3], dtype=F32)
        for k in range(nlev - 1):
            b = bounds[k]
            if np.isfinite(b):
                ts = np.array([b, _below(b)], dtype=F32)
            else:                                   # -inf: every t reaches the level; +inf: none does
                ts = np.array([F32(-3e38), F32(3e38)], dtype=F32)
            acc = np.zeros((1, 2), dtype=np.int32)
            codes = oracle.requantize(acc, np.ones(2, F32), ts, bool(relu), out_bits, out_sign,
                                      res=np.full((1, 2), res_code, np.int8) if has_res else None, res_scale=res_scale,
                                      channel_axis=1).astype(int).reshape(-1)
            level = (codes > 0).astype(int) if out_sign == 2 else codes - qmin
            if np.isfinite(b):
                assert level[0] >= k + 1 and level[1] <= k, (r, k, b, level)
            elif b < 0:
                assert level[0] >= k + 1, (r, k, level)    # e.g. ReLU lifts every t above a signed range's lower levels
            else:
                assert level[1] <= k, (r, k, level)
        assert np.all(np.isinf(bounds[nlev - 1:]))


def test_requant_bounds_refuse_wide_outputs():
    L = lib()
    buf = (ctypes.c_float * 48)()
    assert L.bs_requant_bounds(0, ctypes.c_float(0.0), 0, 0, 1, 3, 0, buf) == 2
    assert L.bs_requant_bounds(0, ctypes.c_float(0.0), 0, 0, 1, 2, 0, None) == 1
