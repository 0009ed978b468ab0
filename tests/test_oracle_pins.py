"""Pins for the CPU oracle: everything here checks oracle/ against facts fixed by the paper's
equations and by mathematics, never against the oracle itself and never against the GPU path."""
import itertools
import os

import numpy as np
import pytest
import torch

import oracle
from oracle import BIPOLAR, SIGNED, UNSIGNED

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _rows(name):
    with open(os.path.join(GOLDEN, name)) as f:
        for line in f:
            line = line.strip()
            if line and not line.startswith("#"):
                yield [c.strip() for c in line.split(";")]


def _rng_codes(rng, shape, bits, sign):
    if sign == BIPOLAR:
        return (2 * rng.integers(0, 2, size=shape) - 1).astype(np.int8)
    lo = -(1 << (bits - 1)) if sign == SIGNED else 0
    hi = (1 << (bits - 1)) - 1 if sign == SIGNED else (1 << bits) - 1
    return rng.integers(lo, hi + 1, size=shape).astype(np.int8)


def _all_codes(bits, sign):
    if sign == BIPOLAR:
        return [-1, 1]
    if sign == SIGNED:
        return list(range(-(1 << (bits - 1)), 1 << (bits - 1)))
    return list(range(1 << bits))


# ---------------------------------------------------------------- worked examples (Section V)

@pytest.mark.parametrize("row", list(_rows("bitserial_dot_worked.txt")), ids=lambda r: r[0])
def test_worked_dot_examples(row):
    name, cfg, a, w, expected = row[0], row[1].split(), row[2].split(), row[3].split(), int(row[4])
    ab, asg, wb, wsg = map(int, cfg)
    a = np.array(a, dtype=np.int8)
    w = np.array(w, dtype=np.int8)
    assert oracle.bitserial_dot(a, w, ab, asg, wb, wsg) == expected          # plane-pair formula
    assert int(oracle.gemm_i32(a[None, :], w[None, :])[0, 0]) == expected    # plain definition
    conv = oracle.conv2d_i32(a.reshape(1, -1, 1, 1), w.reshape(1, -1, 1, 1)) # 1x1 conv on a 1x1 image
    assert int(conv[0, 0, 0, 0]) == expected


# ---------------------------------------------------------------- plane sum == integer dot

SIGN_CASES = [(1, UNSIGNED), (2, UNSIGNED), (2, SIGNED), (1, BIPOLAR)]


@pytest.mark.parametrize("a_cfg", SIGN_CASES)
@pytest.mark.parametrize("w_cfg", SIGN_CASES)
def test_plane_sum_equals_integer_dot_exhaustive(a_cfg, w_cfg):
    """Every operand combination for K <= 3 (and K = 4 for 1-bit operands): the Section V
    plane-pair sum equals sum_k a_k w_k computed here in Python integers."""
    (ab, asg), (wb, wsg) = a_cfg, w_cfg
    av, wv = _all_codes(ab, asg), _all_codes(wb, wsg)
    kmax = 4 if len(av) * len(wv) <= 4 else 3
    for K in range(1, kmax + 1):
        for a in itertools.product(av, repeat=K):
            for w in itertools.product(wv, repeat=K):
                want = sum(x * y for x, y in zip(a, w))
                assert oracle.bitserial_dot(a, w, ab, asg, wb, wsg) == want
                assert int(oracle.gemm_i32(np.array([a]), np.array([w]))[0, 0]) == want


@pytest.mark.parametrize("ab,asg,wb,wsg", [(2, 0, 2, 1), (3, 0, 3, 1), (4, 0, 4, 1), (2, 0, 1, 2), (1, 2, 1, 2),
                                           (3, 1, 2, 1), (4, 1, 1, 0), (1, 0, 3, 0), (1, 2, 3, 1)])
def test_plane_sum_equals_integer_dot_random(ab, asg, wb, wsg):
    rng = np.random.default_rng(11)
    for K in (1, 31, 32, 33, 64, 100):
        a = _rng_codes(rng, K, ab, asg)
        w = _rng_codes(rng, K, wb, wsg)
        want = int(np.dot(a.astype(np.int64), w.astype(np.int64)))
        assert oracle.bitserial_dot(a, w, ab, asg, wb, wsg) == want
        assert int(oracle.gemm_i32(a[None], w[None])[0, 0]) == want


def test_bipolar_xor_identity_exhaustive():
    """dot = K - 2 popcount(a XOR w) for every pair of bipolar vectors up to K = 8."""
    for K in range(1, 9):
        vecs = list(itertools.product((-1, 1), repeat=K))
        step = 1 if K <= 5 else 7
        for a in vecs[::step]:
            for w in vecs[::step]:
                want = sum(x * y for x, y in zip(a, w))
                assert oracle.bipolar_xor_dot(a, w) == want
                assert oracle.bitserial_dot(a, w, 1, BIPOLAR, 1, BIPOLAR) == want
                assert int(oracle.gemm_i32(np.array([a]), np.array([w]))[0, 0]) == want


# ---------------------------------------------------------------- gemm and conv against libraries

def test_gemm_against_int64_matmul():
    rng = np.random.default_rng(3)
    a = _rng_codes(rng, (37, 201), 3, UNSIGNED)
    w = _rng_codes(rng, (19, 201), 3, SIGNED)
    want = a.astype(np.int64) @ w.astype(np.int64).T
    got = oracle.gemm_i32(a, w)
    assert got.dtype == np.int32 and np.array_equal(got, want)
    # a transposed-operand mistake would break this asymmetric case
    assert not np.array_equal(got, (w.astype(np.int64) @ a.astype(np.int64).T).T[:, ::-1])


@pytest.mark.parametrize("k,stride,pad", [(1, 1, 0), (1, 2, 0), (3, 1, 1), (3, 2, 1), (3, 1, 0), (3, 2, 0), (5, 1, 2)])
def test_conv_against_float64_library(k, stride, pad):
    """Integers are exact in float64, so a library convolution is a special-case reference."""
    import torch
    rng = np.random.default_rng(100 + 10 * k + stride + pad)
    N, C, H, W, O = 2, 5, 9, 7, 4
    a = _rng_codes(rng, (N, C, H, W), 2, UNSIGNED)
    w = _rng_codes(rng, (O, C, k, k), 2, SIGNED)
    want = torch.nn.functional.conv2d(torch.from_numpy(a).double(), torch.from_numpy(w).double(),
                                      stride=stride, padding=pad).numpy()
    got = oracle.conv2d_i32(a, w, stride, pad)
    assert got.shape == want.shape
    assert np.array_equal(got.astype(np.float64), want)


def test_conv_border_closed_form():
    """All activations at the top code, all weights +1: each output equals amax * C * (taps that
    fall inside the image): 9 interior, 6 on an edge, 4 in a corner for 3x3 with padding 1."""
    C, H, W, O, amax = 6, 5, 8, 3, 3
    a = np.full((1, C, H, W), amax, dtype=np.int8)
    w = np.ones((O, C, 3, 3), dtype=np.int8)
    got = oracle.conv2d_i32(a, w, 1, 1)
    ty = np.array([2 if y in (0, H - 1) else 3 for y in range(H)])
    tx = np.array([2 if x in (0, W - 1) else 3 for x in range(W)])
    want = amax * C * np.outer(ty, tx)
    for o in range(O):
        assert np.array_equal(got[0, o], want)
    assert got[0, 0, 0, 0] == 4 * amax * C and got[0, 0, 0, 3] == 6 * amax * C and got[0, 0, 2, 3] == 9 * amax * C


def test_conv_single_tap_shifts():
    """A filter with a single 1 at (r, s) copies the input shifted by (r - pad, s - pad): pins the
    tap indexing and the direction of the shift (correlation, not flipped convolution)."""
    rng = np.random.default_rng(5)
    a = _rng_codes(rng, (1, 1, 6, 7), 3, UNSIGNED)
    for r in range(3):
        for s in range(3):
            w = np.zeros((1, 1, 3, 3), dtype=np.int8)
            w[0, 0, r, s] = 1
            got = oracle.conv2d_i32(a, w, 1, 1)[0, 0]
            padded = np.pad(a[0, 0].astype(np.int32), 1)
            want = padded[r:r + 6, s:s + 7]
            assert np.array_equal(got, want)


def test_conv_1x1_stride2_is_gemm_on_subsampled_pixels():
    rng = np.random.default_rng(6)
    N, C, H, W, O = 2, 40, 8, 6, 9
    a = _rng_codes(rng, (N, C, H, W), 2, UNSIGNED)
    w = _rng_codes(rng, (O, C, 1, 1), 2, SIGNED)
    conv = oracle.conv2d_i32(a, w, 2, 0)
    sub = a[:, :, ::2, ::2]
    rows = sub.transpose(0, 2, 3, 1).reshape(-1, C)
    want = (rows.astype(np.int64) @ w.reshape(O, C).astype(np.int64).T).reshape(N, H // 2, W // 2, O).transpose(0, 3, 1, 2)
    assert np.array_equal(conv, want)
    assert np.array_equal(oracle.gemm_i32(rows, w.reshape(O, C)), rows.astype(np.int64) @ w.reshape(O, C).astype(np.int64).T)


def test_conv_channel_and_filter_axes_not_swapped():
    """One nonzero (o, c) weight: only output channel o responds, and only to input channel c."""
    a = np.zeros((1, 3, 2, 2), dtype=np.int8)
    a[0, 2] = 1
    w = np.zeros((4, 3, 1, 1), dtype=np.int8)
    w[1, 2, 0, 0] = -2
    got = oracle.conv2d_i32(a, w)
    assert np.all(got[0, 1] == -2) and np.all(got[0, [0, 2, 3]] == 0)


# ---------------------------------------------------------------- quantiser (Section IV)

@pytest.mark.parametrize("row", list(_rows("quantizer_worked.txt")), ids=lambda r: r[0] + "/" + r[1])
def test_quantizer_worked(row):
    bits, sign = map(int, row[0].split())
    s = float(row[1])
    x = np.array(row[2].split(), dtype=np.float32)
    want = np.array(row[3].split(), dtype=np.int8)
    assert np.array_equal(oracle.quantize(x, s, bits, sign), want)


@pytest.mark.parametrize("bits,sign", [(1, 0), (2, 0), (3, 0), (4, 0), (2, 1), (3, 1), (4, 1)])
def test_quantizer_limits_and_error_bound(bits, sign):
    """Codes stay inside [-Q_N, Q_P] (or [0, 2^b-1]); inside the clip range the reconstruction
    t_hat = t_bar * s is within s/2 of t (quantisation error equation)."""
    rng = np.random.default_rng(bits * 10 + sign)
    s = 0.37
    lo = -(1 << (bits - 1)) if sign else 0
    hi = (1 << (bits - 1)) - 1 if sign else (1 << bits) - 1
    x = rng.uniform((lo - 2) * s, (hi + 2) * s, size=5000).astype(np.float32)
    codes = oracle.quantize(x, s, bits, sign)
    assert codes.min() == lo and codes.max() == hi
    inside = (x >= lo * s) & (x <= hi * s)
    err = np.abs(x.astype(np.float64) - oracle.dequantize(codes, s).astype(np.float64))
    assert np.all(err[inside] <= s / 2 * (1 + 1e-5))
    assert np.all(codes[x > hi * s] == hi) and np.all(codes[x < lo * s] == lo)
    # monotone in x
    order = np.argsort(x)
    assert np.all(np.diff(codes[order].astype(np.int32)) >= 0)


def test_quantizer_bipolar_is_sign():
    x = np.array([-3.0, -0.0, 0.0, 1e-9, 2.0], dtype=np.float32)
    assert np.array_equal(oracle.quantize(x, 1.0, 1, BIPOLAR), np.array([-1, 1, 1, 1, 1], dtype=np.int8))


# ---------------------------------------------------------------- epilogue

@pytest.mark.parametrize("row", list(_rows("epilogue_worked.txt")), ids=lambda r: r[0] + "/" + r[2])
def test_epilogue_worked(row):
    out_bits, out_sign, relu = map(int, row[0].split())
    scale, bias = map(float, row[1].split())
    res_scale = float(row[2])
    acc = np.array(row[3].split(), dtype=np.int32).reshape(1, 1, -1)
    res = None if row[4] == "-" else np.array(row[4].split(), dtype=np.int8).reshape(1, 1, -1)
    want = np.array(row[5].split(), dtype=np.int8)
    got = oracle.requantize(acc, np.array([scale]), np.array([bias]), relu, out_bits, out_sign, res=res, res_scale=res_scale)
    assert np.array_equal(got.reshape(-1), want)


def test_epilogue_per_channel_and_float64_agreement():
    """Each channel uses its own scale/bias; away from rounding ties the fp32 result equals the
    float64 evaluation of clip(round(acc*scale+bias))."""
    rng = np.random.default_rng(9)
    acc = rng.integers(-500, 500, size=(3, 5, 4, 4)).astype(np.int32)
    scale = rng.uniform(0.001, 0.02, 5).astype(np.float32)
    bias = rng.normal(1.5, 1.0, 5).astype(np.float32)
    got = oracle.requantize(acc, scale, bias, True, 2, UNSIGNED)
    v = acc.astype(np.float64) * scale.astype(np.float64)[None, :, None, None] + bias.astype(np.float64)[None, :, None, None]
    v = np.clip(np.maximum(v, 0.0), 0, 3)
    far = np.abs(v - np.floor(v) - 0.5) > 1e-4
    assert far.mean() > 0.99
    assert np.array_equal(got[far], np.rint(v[far]).astype(np.int8))
    assert len(np.unique(got)) == 4
    # gemm layout: channel axis last
    acc2 = rng.integers(-50, 50, size=(7, 5)).astype(np.int32)
    got2 = oracle.requantize(acc2, scale, bias, False, 3, SIGNED, channel_axis=1)
    v2 = np.clip(acc2 * scale.astype(np.float64) + bias.astype(np.float64), -4, 3)
    assert np.array_equal(got2, np.rint(v2).astype(np.int8))


# ---------------------------------------------------------------- storage encodings

@pytest.mark.parametrize("bits,sign", [(1, 0), (2, 0), (3, 0), (4, 0), (2, 1), (3, 1), (1, 2)])
def test_pack_activation_bits_by_definition(bits, sign):
    """Bit (c % 32) of word [n][y][x][c / 32][j] is bit j of the stored pattern of channel c."""
    rng = np.random.default_rng(bits + 7 * sign)
    N, C, H, W = 2, 45, 3, 4
    codes = _rng_codes(rng, (N, C, H, W), bits, sign)
    packed = oracle.pack_activations(codes, bits, sign)
    assert packed.shape == (N, H, W, 2, bits)
    for _ in range(200):
        n, c, y, x, j = (int(rng.integers(0, d)) for d in (N, C, H, W, bits))
        code = int(codes[n, c, y, x])
        pattern = (1 if code > 0 else 0) if sign == BIPOLAR else code & ((1 << bits) - 1)
        assert (int(packed[n, y, x, c // 32, j]) >> (c % 32)) & 1 == (pattern >> j) & 1
    assert np.all(packed[:, :, :, 1, :] >> (C - 32) == 0)          # tail channels are zero
    assert np.array_equal(oracle.unpack_activations(packed, C, bits, sign), codes)


def test_pack_weights_and_rows_by_definition():
    rng = np.random.default_rng(21)
    O, C, R, S, bits = 3, 70, 3, 3, 2
    w = _rng_codes(rng, (O, C, R, S), bits, SIGNED)
    pw = oracle.pack_weights(w, bits, SIGNED)
    assert pw.shape == (O, R, S, 3, bits)
    for _ in range(300):
        o, c, r, s, i = (int(rng.integers(0, d)) for d in (O, C, R, S, bits))
        assert (int(pw[o, r, s, c // 32, i]) >> (c % 32)) & 1 == ((int(w[o, c, r, s]) & 3) >> i) & 1
    rows = _rng_codes(rng, (5, 77), 1, BIPOLAR)
    pr = oracle.pack_rows(rows, 1, BIPOLAR)
    assert pr.shape == (5, 3, 1)
    for m in range(5):
        for k in range(77):
            assert (int(pr[m, k // 32, 0]) >> (k % 32)) & 1 == (1 if rows[m, k] > 0 else 0)
    assert np.all(pr[:, 2, 0] >> (77 - 64) == 0)


def test_popcount_form_on_packed_words_matches_dot():
    """Section V evaluated on the packed words themselves (Python int bit_count on the oracle's
    packed rows) equals the integer matrix product: pins packing and dot product together."""
    rng = np.random.default_rng(33)
    M, N, K, ab, wb = 4, 3, 75, 2, 2
    a = _rng_codes(rng, (M, K), ab, UNSIGNED)
    w = _rng_codes(rng, (N, K), wb, SIGNED)
    pa, pw = oracle.pack_rows(a, ab, UNSIGNED), oracle.pack_rows(w, wb, SIGNED)
    want = a.astype(np.int64) @ w.astype(np.int64).T
    for m in range(M):
        for n in range(N):
            tot = 0
            for i in range(wb):
                for j in range(ab):
                    pc = sum(bin(int(pa[m, kw, j]) & int(pw[n, kw, i])).count("1") for kw in range(pa.shape[1]))
                    tot += (-1 if i == wb - 1 else 1) * (pc << (i + j))
            assert tot == want[m, n]


# ---------------------------------------------------------------- layers kept in floating point

def _fp32_rows():
    for row in _rows("fp32_layers_worked.txt"):
        yield row


@pytest.mark.parametrize("row", list(_fp32_rows()), ids=lambda r: r[0].strip() + ":" + r[1].strip().replace(" ", "x"))
def test_fp32_layers_worked(row):
    kind = row[0].strip()
    f = lambda s: np.array(s.split(), dtype=np.float64).astype(np.float32)
    if kind == "conv":
        C, H, W = map(int, row[1].split())
        O, R, S = map(int, row[2].split())
        stride, pad, relu = map(int, row[3].split())
        got = oracle.conv2d_f32(f(row[4]).reshape(1, C, H, W), f(row[5]).reshape(O, C, R, S), f(row[6]), stride, pad, bool(relu))
        assert np.array_equal(got.reshape(-1), f(row[7]))
    elif kind == "maxpool":
        C, H, W = map(int, row[1].split())
        k, stride, pad = map(int, row[2].split())
        got = oracle.maxpool2d_f32(f(row[3]).reshape(1, C, H, W), k, stride, pad)
        assert np.array_equal(got.reshape(-1), f(row[4]))
    elif kind == "avgpool":
        C, H, W = map(int, row[1].split())
        got = oracle.avgpool_codes(np.array(row[3].split(), dtype=np.int8).reshape(1, C, H, W), float(row[2]))
        assert np.array_equal(got.reshape(-1), f(row[4]))
    else:
        K, J = map(int, row[1].split())
        got = oracle.fc_f32(f(row[2]).reshape(1, K), f(row[3]).reshape(J, K), f(row[4]))
        assert np.array_equal(got.reshape(-1), f(row[5]))


@pytest.mark.parametrize("k,stride,pad", [(7, 2, 3), (3, 1, 1), (1, 1, 0), (5, 2, 0)])
def test_conv_f32_against_float64_library_within_chain_bound(k, stride, pad):
    """A chain of K fused multiply-adds differs from the exact sum by at most K * 2^-24 * sum|x w| (plus the bias term)."""
    rng = np.random.default_rng(k + stride)
    x = rng.normal(0, 1, (2, 3, 19, 23)).astype(np.float32)
    w = rng.normal(0, 0.2, (5, 3, k, k)).astype(np.float32)
    b = rng.normal(0, 1, 5).astype(np.float32)
    got = oracle.conv2d_f32(x, w, b, stride, pad)
    t = lambda a: torch.from_numpy(a.astype(np.float64))
    want = torch.nn.functional.conv2d(t(x), t(w), t(b), stride=stride, padding=pad).numpy()
    mag = torch.nn.functional.conv2d(t(np.abs(x)), t(np.abs(w)), t(np.abs(b)), stride=stride, padding=pad).numpy()
    K = 3 * k * k + 1
    assert np.all(np.abs(got - want) <= K * 2.0 ** -24 * mag)
    assert np.abs(got - want).max() > 0            # binary32 all the way: not a float64 computation rounded at the end
    relu = oracle.conv2d_f32(x, w, b, stride, pad, relu=True)
    assert np.array_equal(relu, np.maximum(got, 0))


def test_conv_f32_single_tap_shift_and_axes():
    """One non-zero weight at (c, r, s) copies a shifted channel: pins the correlation direction, the stride/pad arithmetic
    and the channel / filter axes."""
    rng = np.random.default_rng(3)
    x = rng.normal(0, 1, (2, 3, 9, 11)).astype(np.float32)
    w = np.zeros((4, 3, 3, 3), dtype=np.float32)
    w[2, 1, 0, 2] = 1.0
    got = oracle.conv2d_f32(x, w, None, 2, 1)
    assert not got[:, [0, 1, 3]].any()
    P, Q = got.shape[2:]
    for p in range(P):
        for q in range(Q):
            y, xx = 2 * p - 1 + 0, 2 * q - 1 + 2
            want = x[:, 1, y, xx] if (0 <= y < 9 and 0 <= xx < 11) else 0.0
            assert np.array_equal(got[:, 2, p, q], np.broadcast_to(want, (2,)).astype(np.float32))


def test_pooling_against_library_routines():
    rng = np.random.default_rng(8)
    x = rng.normal(0, 1, (2, 5, 13, 10)).astype(np.float32)
    for k, s, p in ((3, 2, 1), (2, 2, 0), (3, 1, 1)):
        want = torch.nn.functional.max_pool2d(torch.from_numpy(x), k, s, p).numpy()
        assert np.array_equal(oracle.maxpool2d_f32(x, k, s, p), want)
    codes = rng.integers(0, 4, (3, 6, 7, 7)).astype(np.int8)
    inv = np.float32(0.25 / 49)
    want = (codes.astype(np.int64).sum(axis=(2, 3)).astype(np.float32) * inv).astype(np.float32)
    assert np.array_equal(oracle.avgpool_codes(codes, float(inv)), want)
    assert np.allclose(oracle.avgpool_codes(codes, float(inv)), codes.astype(np.float64).mean(axis=(2, 3)) * 0.25, rtol=1e-6)


def test_fc_f32_against_float64_within_chain_bound():
    rng = np.random.default_rng(12)
    x = rng.normal(0, 1, (4, 512)).astype(np.float32)
    w = rng.normal(0, 0.05, (10, 512)).astype(np.float32)
    b = rng.normal(0, 1, 10).astype(np.float32)
    got = oracle.fc_f32(x, w, b)
    want = x.astype(np.float64) @ w.astype(np.float64).T + b.astype(np.float64)
    mag = np.abs(x).astype(np.float64) @ np.abs(w).astype(np.float64).T + np.abs(b)
    assert np.all(np.abs(got - want) <= 513 * 2.0 ** -24 * mag)
