"""`bitserial_gemm_noalloc` against `bitserial_gemm` and against the CPU oracle, through the C ABI.

The no-allocation entry point exists for callers that are not allowed to call cudaMalloc (a host that gave all
device memory to its own pool, an inference loop that must not allocate after start-up, a plugin inside someone
else's stream).  It keeps its scratch in an array built into the library, shared by every call, so the test runs
it several times in a row on different data and on shapes with different split plans.  Outputs must equal the
ordinary entry point's exactly, and both must equal the oracle's integer product and requantised codes (integer
accumulators and packed codes; the GPU tests' tolerance for codes is at most 1e-4 of elements off by one level,
and equality satisfies it).

A call that completes leaves the scratch zero again, so back-to-back calls alone would also pass without the
clearing the entry point does before its kernel.  One case therefore fills the built-in array with a byte
pattern first (the library's test aid), as a predecessor that ended half-way would leave it: only the clearing
makes the call after that exact.

This file is named to be collected last, so a run that stops at the first failure has already run everything else.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2207_08820_b200 import workloads as wl
from paper_2207_08820_b200._lib import lib

pytestmark = pytest.mark.gpu


def _dev(a):
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def _pack_rows(L, codes, bits, sign):
    rows, K = codes.shape
    out = torch.empty(rows * ((K + 31) // 32) * bits, dtype=torch.int32, device="cuda")
    src = _dev(codes)
    assert L.bs_pack_rows(src.data_ptr(), rows, K, bits, sign, out.data_ptr(), None) == 0
    torch.cuda.synchronize()
    return out


def _run(L, fn, ap, wp, M, N, K, scale, bias):
    acc = torch.full((M, N), -7, dtype=torch.int32, device="cuda")
    packed = torch.full((M * ((N + 31) // 32) * 2,), -1, dtype=torch.int32, device="cuda")
    st = fn(ap.data_ptr(), wp.data_ptr(), M, N, K, 2, 0, 1, 2, scale.data_ptr(), bias.data_ptr(), 1, 2, 0,
            acc.data_ptr(), packed.data_ptr(), None)
    assert st == 0, L.bs_status_string(st)
    assert L.bs_check_status(None) == 0
    return acc, packed


def _check_case(L, M, N, K, seed, dirty=None):
    c = wl.gemm_case(M, N, K, seed=seed)
    scale, bias = wl.calibrated_scale_bias(c["w"], 2, 0, 2)
    ap, wp = _pack_rows(L, c["a"], 2, 0), _pack_rows(L, c["w"], 1, 2)
    sc, bi = _dev(scale), _dev(bias)
    want_acc, want_packed = _run(L, L.bitserial_gemm, ap, wp, M, N, K, sc, bi)
    if dirty is not None:
        assert L.bs_selftest_dirty_noalloc_scratch(dirty, None) == 0
    got_acc, got_packed = _run(L, L.bitserial_gemm_noalloc, ap, wp, M, N, K, sc, bi)
    assert torch.equal(got_acc, want_acc)
    assert torch.equal(got_packed, want_packed)
    # and against the oracle: plain integer product, then the epilogue formula and the plane split
    acc = oracle.gemm_i32(c["a"], c["w"])
    assert np.array_equal(got_acc.cpu().numpy(), acc)
    codes = oracle.requantize(acc, scale, bias, True, 2, oracle.UNSIGNED, channel_axis=1)
    assert len(np.unique(codes)) == 4                     # all four levels in use: the epilogue check has teeth
    assert np.array_equal(got_packed.cpu().numpy().view(np.uint32).reshape(M, -1, 2), oracle.pack_rows(codes, 2, oracle.UNSIGNED))
    assert len(np.unique(acc)) > 100                      # a real product, not a constant


def test_noalloc_matches_regular_entry_point_and_oracle_on_calls_in_a_row():
    L = lib()
    assert L.bs_gemm_noalloc_max_scratch_bytes() == 2 * 1024 * 1024
    shapes = [(256, 256, 4608), (256, 256, 4608), (128, 320, 2304), (96, 64, 9216)]   # few output tiles, long reductions
    split = 0
    for k, (M, N, K) in enumerate(shapes):    # calls in a row, different data and plans, same built-in scratch
        need = L.bs_gemm_workspace_bytes(M, N, K, 2, 0, 1, 2)
        assert need <= L.bs_gemm_noalloc_max_scratch_bytes()
        split += need > 0
        _check_case(L, M, N, K, seed=11 + k)
    assert split >= 2                         # the planner really split (and used the scratch for) several of them


@pytest.mark.parametrize("byte", [0xFF, 0x01])
def test_noalloc_clears_a_dirty_scratch(byte):
    """The built-in array is filled with a byte pattern before the call: partial sums would start from garbage and
    the arrival counters would never reach their target unless the entry point cleared what it uses."""
    L = lib()
    M, N, K = 256, 256, 4608
    assert L.bs_gemm_workspace_bytes(M, N, K, 2, 0, 1, 2) > 0
    _check_case(L, M, N, K, seed=21, dirty=byte)
    _check_case(L, M, N, K, seed=22)          # and an undisturbed call right after it


def test_noalloc_rejects_shapes_beyond_the_builtin_scratch():
    L = lib()
    M, N, K = 768, 768, 18432                 # the split plan of this shape wants about 2.3 MB of scratch
    need = L.bs_gemm_workspace_bytes(M, N, K, 2, 0, 1, 2)
    if need <= L.bs_gemm_noalloc_max_scratch_bytes():
        M, N, K = 1024, 768, 73728
        need = L.bs_gemm_workspace_bytes(M, N, K, 2, 0, 1, 2)
    if need <= L.bs_gemm_noalloc_max_scratch_bytes():
        pytest.skip("no oversized split plan found for the probe shapes")
    buf = torch.zeros(16, dtype=torch.int32, device="cuda")   # never dereferenced: the call is refused on the host
    st = L.bitserial_gemm_noalloc(buf.data_ptr(), buf.data_ptr(), M, N, K, 2, 0, 1, 2, None, None, 0, 0, 0,
                                  buf.data_ptr(), None, None)
    assert st == 2                                            # BS_ERR_UNSUPPORTED
