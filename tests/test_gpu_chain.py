"""GPU parity of ``bitserial_conv2d_tc_chain`` (several same-shaped layers in one launch): every layer's packed output against
the oracle run layer by layer on the same seeded inputs (direct integer convolution + requantisation), word for word; repeated
launches on one workspace, CUDA-graph replay, guard words around every output, and the shapes the entry point must refuse."""
import ctypes

import numpy as np
import pytest
import torch

import oracle
from paper_2207_08820_b200 import api, workloads as wl
from paper_2207_08820_b200._lib import lib
from paper_2207_08820_b200.net import BitserialNet
from gpu_util import Guarded, dev, words

pytestmark = pytest.mark.gpu

A_BITS, W_BITS = 2, 2


def make_chain(seed, N, C, H, W, k, nlayers, res_scale=0.75, a_bits=A_BITS):
    """Seeded layers shaped like consecutive residual blocks: layer l reads layer l - 1; odd layers add the input of their block
    (the chain's input for layer 1, the output of layer 1 for layer 3).  Scale and bias are set from the oracle's accumulators
    so that all four codes occur.  Returns the input codes, the per-layer dicts and the oracle's codes per layer."""
    rng = np.random.default_rng(seed)
    top = (1 << a_bits) - 1
    x = rng.integers(0, top + 1, size=(N, C, H, W), dtype=np.int8)
    layers, want = [], []
    cur, block_in = x, x
    for l in range(nlayers):
        w = rng.integers(-2, 2, size=(C, C, k, k), dtype=np.int8)
        acc = oracle.conv2d_i32(cur, w, stride=1, pad=k // 2)
        sd = float(acc.std()) + 1.0
        scale = (rng.uniform(0.8, 1.6, size=C) * (top / 3.0) / sd).astype(np.float32)
        bias = (top / 2.0 - acc.mean(axis=(0, 2, 3)) * scale + rng.normal(0, 0.3, size=C)).astype(np.float32)
        res = block_in if l % 2 == 1 else None
        if res is not None:
            bias -= np.float32(res_scale * top / 2.0)
        codes = oracle.requantize(acc, scale, bias, True, a_bits, oracle.UNSIGNED, res=res, res_scale=res_scale if res is not None else 0.0)
        layers.append(dict(w=w, scale=scale, bias=bias, res=(-1 if l == 1 else l - 2) if res is not None else None,
                           res_scale=res_scale if res is not None else 0.0))
        want.append(codes)
        if l % 2 == 1:
            block_in = codes
        cur = codes
    return x, layers, want


class ChainOnGpu:
    def __init__(self, x, layers, k, a_bits=A_BITS):
        N, C, H, W = x.shape
        self.k, self.C, self.a_bits = k, C, a_bits
        self.guard = Guarded()
        self.x = api.bitpack_activations(dev(x.astype(np.float32)), 1.0, a_bits, api.UNSIGNED, api.NCHW)
        self.x = self.x.view(N, H, W, C // 32, a_bits)
        self.outs = [self.guard.empty((N, H, W, C // 32, a_bits), fill=-1) for _ in layers]
        self.wp, self.wtc, self.params, self.acts, self.keep = [], [], [], [], []
        for l, L in enumerate(layers):
            wp = api.pack_weights(dev(L["w"]), W_BITS, api.SIGNED)
            self.wp.append(wp)
            self.wtc.append(api.tc_prepare_weights(wp, C, api.SIGNED, a_bits))
            act = self.x if l == 0 else self.outs[l - 1]
            res = None if L["res"] is None else (self.x if L["res"] < 0 else self.outs[L["res"]])
            scale, bias = dev(L["scale"]), dev(L["bias"])
            self.keep += [scale, bias]
            self.acts.append(act)
            self.params.append(api.conv_params(act.shape, wp.shape, C=C, stride=1, pad=k // 2, a_sign=api.UNSIGNED, w_sign=api.SIGNED,
                                               scale=scale, bias=bias, relu=True, out_bits=a_bits, out_sign=api.UNSIGNED, residual=res,
                                               res_scale=L["res_scale"], res_bits=a_bits if res is not None else 0, res_sign=api.UNSIGNED))
        self.nbytes = api.tc_chain_workspace_bytes(self.params)
        self.ws = torch.zeros(max(self.nbytes, 4) // 4, dtype=torch.int32, device="cuda")
        torch.cuda.synchronize()

    def run(self):
        api.bitserial_conv2d_tc_chain(self.acts, self.wtc, self.params, self.outs, self.ws)

    def check(self, want):
        api.bs_check_status()
        self.guard.check()
        for l, codes in enumerate(want):
            got = words(self.outs[l]).reshape(-1)
            ref = oracle.pack_activations(codes, self.a_bits, oracle.UNSIGNED).reshape(-1)
            assert np.array_equal(got, ref), f"layer {l}: {(got != ref).sum()} of {ref.size} words differ"


SHAPES = [
    # seed, N, C, H, W, k, layers
    (11, 3, 64, 24, 24, 3, 4),
    (12, 5, 128, 14, 14, 3, 3),
    (13, 8, 64, 56, 56, 3, 4),       # 224 pixel tiles per layer over several hundred CTAs: tiles really wait for other CTAs
    (14, 2, 64, 20, 12, 5, 2),
    (15, 4, 64, 16, 16, 1, 2),       # 1x1: flat pixel tiles
    (16, 1, 32, 40, 40, 3, 2),
    (17, 6, 128, 28, 28, 3, 3),
    (18, 2, 64, 9, 11, 3, 3),        # ragged: tiles hang over the image on both axes
]


@pytest.mark.parametrize("seed,N,C,H,W,k,nlayers", SHAPES)
def test_chain_matches_oracle(seed, N, C, H, W, k, nlayers):
    x, layers, want = make_chain(seed, N, C, H, W, k, nlayers)
    levels = set(np.unique(want[-1]).tolist())
    assert len(levels) >= 3                   # the seeded layers do not collapse to a constant
    g = ChainOnGpu(x, layers, k)
    if g.nbytes == 0:
        pytest.skip("the planner does not run this shape with resident filters")
    g.run()
    g.check(want)


@pytest.mark.parametrize("a_bits", [1, 3, 4])
def test_chain_other_activation_widths(a_bits):
    """The 1-, 3- and 4-bit instantiations of the chain kernel (3- and 4-bit outputs take the formula epilogue, 4-bit records are
    twice as long): same comparison with the oracle, layer by layer."""
    x, layers, want = make_chain(30 + a_bits, 3, 64, 24, 24, 3, 3, a_bits=a_bits)
    assert len(np.unique(want[-1])) >= min(3, 1 << a_bits)
    g = ChainOnGpu(x, layers, 3, a_bits=a_bits)
    if g.nbytes == 0:
        pytest.skip("the tensor-core path does not take this activation width at this shape")
    g.run()
    g.check(want)


def test_chain_repeated_launches_and_graph_replay():
    """The progress counters live on from launch to launch: three launches in a row, then a captured graph replayed three
    times, with the outputs wiped in between; every run must reproduce the oracle."""
    x, layers, want = make_chain(21, 4, 64, 28, 28, 3, 4)
    g = ChainOnGpu(x, layers, 3)
    assert g.nbytes > 0
    for _ in range(3):
        for o in g.outs:
            o.fill_(-1)
        g.run()
        g.check(want)
    stream = torch.cuda.Stream()
    with torch.cuda.stream(stream):
        g.run()
        stream.synchronize()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=stream):
            g.run()
        for _ in range(3):
            for o in g.outs:
                o.fill_(-1)
            graph.replay()
            stream.synchronize()
            g.check(want)


def test_chain_equals_layer_by_layer_entry_point():
    x, layers, want = make_chain(22, 2, 64, 32, 32, 3, 4)
    g = ChainOnGpu(x, layers, 3)
    assert g.nbytes > 0
    g.run()
    g.check(want)
    chain_out = [o.clone() for o in g.outs]
    for o in g.outs:
        o.fill_(-1)
    for l, L in enumerate(layers):
        res = None if L["res"] is None else (g.x if L["res"] < 0 else g.outs[L["res"]])
        api.bitserial_conv2d(g.acts[l], g.wp[l], C=g.C, stride=1, pad=1, scale=g.keep[2 * l], bias=g.keep[2 * l + 1], relu=True,
                             out_bits=A_BITS, residual=res, res_scale=L["res_scale"], res_bits=A_BITS if res is not None else 0,
                             out_packed=g.outs[l], wgt_tc=g.wtc[l])
    api.bs_check_status()
    for a, b in zip(chain_out, g.outs):
        assert torch.equal(a, b)


def test_chain_refuses_what_it_cannot_run():
    x, layers, _ = make_chain(23, 2, 64, 16, 16, 3, 2)
    g = ChainOnGpu(x, layers, 3)
    assert g.nbytes > 0
    L = lib()
    n = 2
    vp = ctypes.c_void_p * n
    arr = (type(g.params[0]) * n)(*g.params)

    def call(acts, outs, params=arr, ws=g.ws, nbytes=None):
        return L.bitserial_conv2d_tc_chain(n, vp(*[t.data_ptr() for t in acts]), vp(*[t.data_ptr() for t in g.wtc]), params,
                                           vp(*[t.data_ptr() for t in outs]), ws.data_ptr(), g.ws.numel() * 4 if nbytes is None else nbytes,
                                           0, None)

    assert call(g.acts, g.outs) == 0
    assert call(g.acts, g.outs, nbytes=16) == 1                         # workspace too small
    assert call(g.acts, [g.outs[0], g.outs[0]]) == 2                    # layer 1 would read what it writes
    assert call([g.outs[1], g.outs[0]], g.outs) == 2                    # layer 0 would read a later layer's output
    # a stride-2 layer, layers of different widths, a single layer, five layers: no chain
    bad = (type(g.params[0]) * n)(*g.params)
    bad[1].stride = 2
    assert L.bs_tc_chain_workspace_bytes(bad, n) == 0
    assert call(g.acts, g.outs, params=bad) == 2
    bad = (type(g.params[0]) * n)(*g.params)
    bad[1].O = 128
    assert L.bs_tc_chain_workspace_bytes(bad, n) == 0
    assert L.bs_tc_chain_workspace_bytes(arr, 1) == 0
    assert L.bs_tc_chain_workspace_bytes(arr, 5) == 0
    torch.cuda.synchronize()
    api.bs_check_status()


def test_net_runner_uses_chains_and_fewer_launches():
    net = wl.resnet18_body(4)
    params = wl.network_params(net, 3000)
    runner = BitserialNet(net, params, 0.25, batch=4, engine="tc", chains=True)
    plain = BitserialNet(net, params, 0.25, batch=4, engine="tc", chains=False)
    assert len(plain.units) == len(net.layers) == 19
    assert len(runner.units) < 19
    assert max(len(u["items"]) for u in runner.units) >= 3
    x = dev(wl.network_input(net, 3000, 0.25, batch=4))
    a = runner.forward(x).clone()
    b = plain.forward(x).clone()
    api.bs_check_status()
    assert torch.equal(a, b)
    for name in net.tensor_shapes():
        assert torch.equal(runner.bufs[name], plain.bufs[name]), name
    # "auto" keeps, per run of layers, whichever form it timed faster: any mix of the two, same results
    auto = BitserialNet(net, params, 0.25, batch=4, engine="tc", chains="auto")
    assert len(runner.units) <= len(auto.units) <= 19
    assert torch.equal(auto.forward(x), b)
    api.bs_check_status()
