"""Runs a stack of quantised conv layers (``workloads.NetSpec``) through the C ABI.

Host logic only: buffer planning, weight packing at set-up, one ``bitserial_conv2d`` call per layer
(residual adds and concatenations are epilogue arguments), optional CUDA-graph replay.
"""
from __future__ import annotations

from typing import Dict, Optional

import numpy as np
import torch

from . import api
from .workloads import NetSpec


class BitserialNet:
    def __init__(self, net: NetSpec, params: Dict[str, Dict], act_scale: float, device="cuda", batch: Optional[int] = None,
                 engine: str = "popc", concurrent: bool = True):
        """engine: "popc" = popcount kernels on the integer pipes; "tc" = tensor-core entry point for every layer it
        supports (others fall back to the popcount kernel).  concurrent: launch independent neighbouring layers on
        two streams (see :meth:`run_layers`)."""
        self.net = net
        self.engine = engine
        self.act_scale = float(act_scale)
        self.device = torch.device(device)
        self.batch = batch or net.batch
        self.shapes = net.tensor_shapes()
        self.layers = []
        for L in net.layers:
            p = params[L.name]
            w = torch.from_numpy(np.ascontiguousarray(p["w"])).to(self.device)
            wp = api.pack_weights(w, net.w_bits, p["w_sign"])
            _, H, W = self.shapes[L.src]
            use_tc = engine == "tc" and api.tc_supported(self.batch, L.C, H, W, L.O, L.k, L.stride, L.pad, net.a_bits,
                                                         api.UNSIGNED, net.w_bits, p["w_sign"])
            self.layers.append(dict(
                spec=L,
                w=wp,
                w_tc=api.tc_prepare_weights(wp, L.C, p["w_sign"], net.a_bits) if use_tc else None,
                w_sign=p["w_sign"],
                scale=torch.from_numpy(p["scale"]).to(self.device),
                bias=torch.from_numpy(p["bias"]).to(self.device)))
        self.bufs: Dict[str, torch.Tensor] = {}
        for name, (C, H, W) in self.shapes.items():
            self.bufs[name] = torch.zeros(self.batch, H, W, (C + 31) // 32, net.a_bits, dtype=torch.int32, device=self.device)
        torch.cuda.synchronize(self.device)   # chained layers fetch filters, scale and bias ahead of stream order
        self.concurrent = concurrent
        self.side = torch.cuda.Stream(device=self.device)
        self.graph = None
        self.static_in = None
        self.launches_per_forward = 2 + len(self.layers)

    def _run(self, x: torch.Tensor) -> torch.Tensor:
        self.pack_input(x)
        self.run_layers()
        return self.bufs[self.net.out_name]

    def pack_input(self, x: torch.Tensor) -> None:
        """Quantise + bitplane-pack the fp32 input on the current stream; the filter prefetch runs beside it on the
        side stream (a fork and a join: two parallel nodes under stream capture)."""
        net = self.net
        main = torch.cuda.current_stream(self.device)
        fork = torch.cuda.Event()
        fork.record(main)
        self.side.wait_event(fork)
        with torch.cuda.stream(self.side):
            self.prefetch_filters()
            done = torch.cuda.Event()
            done.record(self.side)
        api.bitpack_activations(x, self.act_scale, net.a_bits, api.UNSIGNED, api.NCHW, out=self.bufs[net.in_name].view(-1))
        main.wait_event(done)

    def run_layer(self, item, chained: bool = True) -> None:
        """One conv layer through the C ABI on the current stream."""
        net, L = self.net, item["spec"]
        res = self.bufs[L.res] if L.res else None
        api.bitserial_conv2d(
            self.bufs[L.src], item["w"], C=L.C, stride=L.stride, pad=L.pad, a_sign=api.UNSIGNED,
            w_sign=item["w_sign"], scale=item["scale"], bias=item["bias"], relu=L.relu, out_bits=net.a_bits,
            out_sign=api.UNSIGNED, residual=res, res_scale=L.res_scale, res_bits=net.a_bits if L.res else 0,
            res_sign=api.UNSIGNED, res_c_offset=0, res_c_total=self.shapes[L.res][0] if L.res else 0,
            out_packed=self.bufs[L.dst], out_c_offset=L.dst_c_offset, out_c_total=self.shapes[L.dst][0],
            wgt_tc=item["w_tc"], chained=chained and item["w_tc"] is not None)

    def run_layers(self) -> None:
        """All conv layers in order.  With ``concurrent`` a layer whose successor in the list neither reads nor
        overwrites its output (a projection shortcut beside the first conv of its block, the two 1x1 branches of a
        cross-stage block) is launched on a side stream, so the two kernels share the GPU; events carry the
        dependencies, and under stream capture they become the edges of the graph."""
        main = torch.cuda.current_stream(self.device)
        pending: Dict[str, torch.cuda.Event] = {}
        n = len(self.layers)
        for i, item in enumerate(self.layers):
            L = item["spec"]
            nxt = self.layers[i + 1]["spec"] if i + 1 < n else None
            aside = (self.concurrent and nxt is not None and L.dst not in (nxt.src, nxt.res)
                     and nxt.dst not in (L.src, L.res)
                     and (nxt.dst != L.dst or nxt.dst_c_offset != L.dst_c_offset) and L.src not in pending
                     and (L.res is None or L.res not in pending))
            if aside:
                fork = torch.cuda.Event()
                fork.record(main)
                self.side.wait_event(fork)
                with torch.cuda.stream(self.side):
                    self.run_layer(item, chained=False)
                    done = torch.cuda.Event()
                    done.record(self.side)
                pending[L.dst] = done
                continue
            for t in (L.src, L.res, L.dst):
                if t is not None and t in pending:
                    main.wait_event(pending.pop(t))
            self.run_layer(item)
        for ev in pending.values():
            main.wait_event(ev)

    def prefetch_filters(self) -> None:
        """The filters of every layer start on their way into L2 while the pack kernel and the first layers run."""
        api.l2_prefetch([item["w_tc"] if item["w_tc"] is not None else item["w"] for item in self.layers])

    def forward(self, x: torch.Tensor) -> torch.Tensor:
        """x: float32 [batch, C, H, W] on the device.  Returns the packed output tensor of the stack."""
        return self._run(x)

    def capture(self, x: torch.Tensor) -> None:
        """Record one forward pass into a CUDA graph replayed by :meth:`replay` (input copied into a static buffer)."""
        self.static_in = x.clone()
        self._run(self.static_in)            # warm-up outside capture: plans, descriptors, module loading
        torch.cuda.synchronize()
        self.graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(self.graph):
            self._run(self.static_in)

    def replay(self, x: Optional[torch.Tensor] = None) -> torch.Tensor:
        if x is not None:
            self.static_in.copy_(x, non_blocking=True)
        self.graph.replay()
        return self.bufs[self.net.out_name]

    def unpacked(self, name: str) -> torch.Tensor:
        """int8 NCHW codes of an activation tensor (debugging / tests)."""
        C = self.shapes[name][0]
        return api.bitunpack_activations(self.bufs[name], C, self.net.a_bits, api.UNSIGNED, api.NCHW)


class BitserialFullNet:
    """The whole mixed-precision classifier of ``workloads.FullNetSpec`` through the C ABI: floating-point stem
    (``bs_conv2d_f32`` + ``bs_maxpool2d_f32``), quantise + pack, the quantised body (:class:`BitserialNet`), floating-point head
    (``bs_avgpool_codes_f32`` + ``bs_fc_f32``).  Host logic only."""

    def __init__(self, net, params: Dict[str, Dict], device="cuda", batch: Optional[int] = None, engine: str = "tc"):
        self.net = net
        self.batch = batch or net.batch
        self.device = torch.device(device)
        self.body = BitserialNet(net.body, params, net.stem_act_scale, device=device, batch=self.batch, engine=engine)
        to = lambda a: torch.from_numpy(np.ascontiguousarray(a)).to(self.device)
        self.stem_w, self.stem_b = to(params["stem"]["w"]), to(params["stem"]["bias"])
        self.fc_w, self.fc_b = to(params["fc"]["w"]), to(params["fc"]["bias"])
        h1 = (net.hw + 2 * 3 - 7) // 2 + 1
        h2 = (h1 + 2 - 3) // 2 + 1
        self.stem_conv = torch.empty(self.batch, 64, h1, h1, dtype=torch.float32, device=self.device)
        self.stem_pool = torch.empty(self.batch, 64, h2, h2, dtype=torch.float32, device=self.device)
        C, H, W = net.body.tensor_shapes()[net.body.out_name]
        self.pooled = torch.empty(self.batch, C, dtype=torch.float32, device=self.device)
        self.logits = torch.empty(self.batch, net.classes, dtype=torch.float32, device=self.device)
        self.inv = float(np.float32(np.float32(net.body_act_scale) / np.float32(H * W)))
        self.launches_per_forward = 4 + self.body.launches_per_forward

    def run_stem(self, images: torch.Tensor) -> None:
        api.conv2d_f32(images, self.stem_w, self.stem_b, stride=2, pad=3, relu=True, out=self.stem_conv)
        api.maxpool2d_f32(self.stem_conv, 3, 2, 1, out=self.stem_pool)

    def run_head(self) -> None:
        body = self.net.body
        api.avgpool_codes_f32(self.body.bufs[body.out_name], body.tensor_shapes()[body.out_name][0], api.UNSIGNED, self.inv, out=self.pooled)
        api.fc_f32(self.pooled, self.fc_w, self.fc_b, out=self.logits)

    def forward(self, images: torch.Tensor) -> torch.Tensor:
        """images: float32 [batch, 3, hw, hw] on the device.  Returns the logits [batch, classes]."""
        self.run_stem(images)
        self.body.pack_input(self.stem_pool)
        self.body.run_layers()
        self.run_head()
        return self.logits
