"""Host-only checks of the C ABI: the library loads without a GPU, exports every symbol the header
declares, agrees with the header on struct layout and size formulas, and rejects bad arguments on
the host before touching a device."""
import ctypes
import os
import re
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
HEADER = os.path.join(ROOT, "include", "bitserial.h")


@pytest.fixture(scope="module")
def L():
    from paper_2207_08820_b200 import build
    build.build()
    from paper_2207_08820_b200 import _lib
    return _lib.lib()


def _declared_functions():
    src = open(HEADER).read()
    src = re.sub(r"/\*.*?\*/", "", src, flags=re.S)
    names = re.findall(r"^\s*(?:int|size_t|const char\*)\s+(\w+)\s*\(", src, flags=re.M)
    return sorted(set(names))


def test_every_declared_symbol_is_exported(L):
    names = _declared_functions()
    assert {"bitpack_activations", "pack_weights", "bitserial_conv2d", "bitserial_gemm"} <= set(names)
    for n in names:
        assert hasattr(L, n), n


def test_header_compiles_as_c_and_struct_matches_binding(tmp_path):
    from paper_2207_08820_b200._lib import ConvParams
    src = tmp_path / "t.c"
    src.write_text('#include <stdio.h>\n#include <stddef.h>\n#include "bitserial.h"\n'
                   'int main(void){printf("%zu %zu %zu %zu %zu\\n", sizeof(bs_conv_params), offsetof(bs_conv_params, scale),'
                   ' offsetof(bs_conv_params, residual), offsetof(bs_conv_params, res_scale), offsetof(bs_conv_params, i32_layout));return 0;}\n')
    exe = tmp_path / "t"
    subprocess.run(["gcc", "-std=c99", "-Wall", "-Werror", "-I", os.path.join(ROOT, "include"), str(src), "-o", str(exe)], check=True)
    out = subprocess.run([str(exe)], capture_output=True, text=True, check=True).stdout.split()
    assert int(out[0]) == ctypes.sizeof(ConvParams)
    assert int(out[1]) == ConvParams.scale.offset
    assert int(out[2]) == ConvParams.residual.offset
    assert int(out[3]) == ConvParams.res_scale.offset
    assert int(out[4]) == ConvParams.i32_layout.offset


def test_size_queries(L):
    assert L.bs_packed_act_bytes(1, 64, 56, 56, 2) == 56 * 56 * 2 * 2 * 4
    assert L.bs_packed_act_bytes(2, 33, 3, 5, 3) == 2 * 3 * 5 * 2 * 3 * 4
    assert L.bs_packed_wgt_bytes(64, 64, 3, 3, 2) == 64 * 9 * 2 * 2 * 4
    assert L.bs_packed_rows_bytes(10, 577, 1) == 10 * 19 * 4
    assert L.bs_packed_act_bytes(1, 64, 56, 56, 5) == 0
    assert L.bs_packed_wgt_bytes(0, 64, 3, 3, 2) == 0


def test_bad_arguments_are_rejected_on_the_host(L):
    from paper_2207_08820_b200._lib import ConvParams
    buf = (ctypes.c_char * 4096)()
    addr = (ctypes.addressof(buf) + 255) & ~255      # never dereferenced: validation fails first
    INVALID, UNSUPPORTED, ALIGN = 1, 2, 3
    assert L.bitpack_activations(None, 1, 0, 1, 64, 8, 8, 1.0, 2, 0, addr, None) == INVALID
    assert L.bitpack_activations(addr, 1, 0, 1, 64, 8, 8, 1.0, 5, 0, addr, None) == INVALID
    assert L.bitpack_activations(addr, 1, 0, 1, 64, 8, 8, 1.0, 2, 2, addr, None) == INVALID      # bipolar needs 1 bit
    assert L.bitpack_activations(addr, 1, 0, 1, 64, 8, 8, 0.0, 2, 0, addr, None) == INVALID      # scale must be > 0
    assert L.bitpack_activations(addr + 4, 1, 0, 1, 64, 8, 8, 1.0, 2, 0, addr, None) == ALIGN
    assert L.pack_weights(addr, 0, 64, 64, 3, 3, 0, 1, addr, None) == INVALID
    p = ConvParams(N=1, C=64, H=8, W=8, O=64, R=3, S=3, stride=1, pad=1, a_bits=2, a_sign=0, w_bits=2, w_sign=1,
                   i32_layout=0)
    assert L.bitserial_conv2d(addr, addr, ctypes.byref(p), None, None, None) == INVALID          # no output
    p.R = 3; p.S = 1
    assert L.bitserial_conv2d(addr, addr, ctypes.byref(p), addr, None, None) == UNSUPPORTED
    p.S = 3; p.stride = 3
    assert L.bitserial_conv2d(addr, addr, ctypes.byref(p), addr, None, None) == UNSUPPORTED
    p.stride = 1; p.a_bits = 1; p.a_sign = 2
    assert L.bitserial_conv2d(addr, addr, ctypes.byref(p), addr, None, None) == UNSUPPORTED      # bipolar acts with padding
    p.a_bits = 2; p.a_sign = 0
    assert L.bitserial_conv2d(addr, addr, ctypes.byref(p), None, addr, None) == INVALID          # packed output needs scale/bias
    assert L.bitserial_conv2d(addr, addr + 8, ctypes.byref(p), addr, None, None) == ALIGN
    p.C = 1 << 28                                                                                 # accumulator could overflow
    p.a_bits = 4; p.w_bits = 4
    assert L.bitserial_conv2d(addr, addr, ctypes.byref(p), addr, None, None) == UNSUPPORTED
    assert L.bitserial_gemm(addr, addr, 0, 4, 4, 2, 0, 2, 1, None, None, 0, 0, 0, addr, None, None) == INVALID
    assert L.bs_status_string(5) == b"BS_ERR_TIMEOUT"
    assert L.bs_selftest_wait_timeout(0, None) == INVALID          # refused before any launch
    assert L.bs_selftest_wait_timeout(1 << 20, None) == INVALID
    # bs_l2_prefetch: nothing to do is fine; missing arrays, null or misaligned buffers are refused before any launch
    assert L.bs_l2_prefetch(None, None, 0, None) == 0
    assert L.bs_l2_prefetch(None, None, 1, None) == INVALID
    ptrs = (ctypes.c_void_p * 2)(addr, None)
    sizes = (ctypes.c_size_t * 2)(256, 256)
    assert L.bs_l2_prefetch(ptrs, sizes, 2, None) == INVALID
    ptrs[1] = addr + 8
    assert L.bs_l2_prefetch(ptrs, sizes, 2, None) == ALIGN
    # tensor-core entry points: channel counts and pixel records the tensor-core path cannot take
    p2 = ConvParams(N=1, C=40, H=8, W=8, O=64, R=3, S=3, stride=1, pad=1, a_bits=2, a_sign=0, w_bits=2, w_sign=1, i32_layout=0)
    assert L.bs_tc_supported(ctypes.byref(p2)) == 0
    assert L.bitserial_conv2d_tc(addr, addr, ctypes.byref(p2), addr, None, None) == UNSUPPORTED
    assert L.bitserial_conv2d_tc_chained(addr, addr, ctypes.byref(p2), addr, None, None) == UNSUPPORTED
    assert L.bs_tc_weights_bytes(64, 40, 3, 3) == 0
    assert L.bs_tc_weights_bytes(200, 64, 3, 3) == 256 * 9 * 64


def test_chain_query_and_refusals_on_the_host(L):
    """The chain planner answers without a device (it plans for a full B200): same-shaped stride-1 layers with packed outputs
    are accepted, anything else gives 0 bytes, and the launch entry point refuses bad arguments before touching the GPU."""
    from paper_2207_08820_b200._lib import ConvParams
    buf = (ctypes.c_char * 4096)()
    addr = (ctypes.addressof(buf) + 255) & ~255      # stands for device pointers; never dereferenced on these paths
    INVALID, UNSUPPORTED = 1, 2

    def layer(**kw):
        d = dict(N=8, C=64, H=56, W=56, O=64, R=3, S=3, stride=1, pad=1, a_bits=2, a_sign=0, w_bits=2, w_sign=1, scale=addr, bias=addr,
                 relu=1, out_bits=2, out_sign=0, out_c_offset=0, out_c_total=64, i32_layout=0)
        d.update(kw)
        return ConvParams(**d)

    def arr(*layers):
        a = (ConvParams * len(layers))()
        for k, q in enumerate(layers):
            ctypes.memmove(ctypes.addressof(a[k]), ctypes.addressof(q), ctypes.sizeof(ConvParams))
        return a

    four = arr(layer(), layer(residual=addr, res_bits=2, res_scale=0.5, res_c_total=64), layer(), layer())
    nbytes = L.bs_tc_chain_workspace_bytes(four, 4)
    tiles = 8 * 4 * 7                                   # 56 x 56 in tiles of 16 x 8 pixels
    assert nbytes == (4 * tiles + 4) * 4
    assert L.bs_tc_chain_workspace_bytes(four, 2) == (2 * tiles + 4) * 4
    assert L.bs_tc_chain_workspace_bytes(four, 1) == 0 and L.bs_tc_chain_workspace_bytes(four, 5) == 0
    assert L.bs_tc_chain_workspace_bytes(None, 2) == 0
    assert L.bs_tc_chain_workspace_bytes(arr(layer(), layer(stride=2)), 2) == 0            # output smaller than input
    assert L.bs_tc_chain_workspace_bytes(arr(layer(), layer(O=128, out_c_total=128)), 2) == 0
    assert L.bs_tc_chain_workspace_bytes(arr(layer(), layer(R=1, S=1, pad=0)), 2) == 0     # kernel sizes differ
    assert L.bs_tc_chain_workspace_bytes(arr(layer(out_bits=3), layer()), 2) == 0          # next layer reads 2-bit activations
    assert L.bs_tc_chain_workspace_bytes(arr(layer(out_bits=0), layer()), 2) == 0          # a layer without packed output
    assert L.bs_tc_chain_workspace_bytes(arr(layer(out_c_total=96), layer()), 2) == 0      # output is a slice of a wider tensor
    vp = ctypes.c_void_p * 2
    two = arr(layer(), layer())
    ptrs = vp(addr, addr + 1024)
    assert L.bitserial_conv2d_tc_chain(2, None, ptrs, two, ptrs, addr, 1 << 20, 0, None) == INVALID
    assert L.bitserial_conv2d_tc_chain(2, ptrs, ptrs, two, ptrs, None, 1 << 20, 0, None) == INVALID
    assert L.bitserial_conv2d_tc_chain(2, vp(addr, None), ptrs, two, ptrs, addr, 1 << 20, 0, None) == INVALID
    assert L.bitserial_conv2d_tc_chain(1, ptrs, ptrs, two, ptrs, addr, 1 << 20, 0, None) == UNSUPPORTED
    assert L.bitserial_conv2d_tc_chain(5, ptrs, ptrs, two, ptrs, addr, 1 << 20, 0, None) == UNSUPPORTED


def test_binding_fails_loudly_without_library(tmp_path):
    """Importing the binding with the shared library absent must raise, not fall back."""
    code = ("import sys; sys.path.insert(0, %r)\n"
            "from paper_2207_08820_b200 import _lib\n"
            "_lib.LIB_PATH = %r\n"
            "try:\n    _lib.lib()\nexcept ImportError as e:\n    print('RAISED'); sys.exit(0)\nsys.exit(1)\n"
            % (ROOT, str(tmp_path / "nope.so")))
    r = subprocess.run([sys.executable, "-c", code], capture_output=True, text=True)
    assert r.returncode == 0 and "RAISED" in r.stdout


def test_product_never_imports_oracle():
    pkg = os.path.join(ROOT, "paper_2207_08820_b200")
    for dirpath, _, files in os.walk(pkg):
        if "_build" in dirpath:
            continue
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".h")):
                text = open(os.path.join(dirpath, f)).read()
                assert "import oracle" not in text and "from oracle" not in text and "bitserial_oracle" not in text, f
