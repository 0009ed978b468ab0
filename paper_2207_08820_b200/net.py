"""Runs a stack of quantised conv layers (``workloads.NetSpec``) through the C ABI.

Host logic only: buffer planning, weight packing at set-up, one ``bitserial_conv2d`` call per layer -- or one
``bitserial_conv2d_tc_chain`` call per run of same-shaped layers -- (residual adds and concatenations are epilogue
arguments), optional CUDA-graph replay.
"""
from __future__ import annotations

from typing import Dict, List, Optional

import numpy as np
import torch

from . import api
from .workloads import NetSpec


class BitserialNet:
    MAX_CHAIN = 4

    def __init__(self, net: NetSpec, params: Dict[str, Dict], act_scale: float, device="cuda", batch: Optional[int] = None,
                 engine: str = "popc", concurrent: bool = True, chains="auto"):
        """engine: "popc" = popcount kernels on the integer pipes; "tc" = tensor-core entry point for every layer it
        supports (others fall back to the popcount kernel).  concurrent: launch independent neighbouring layers on
        two streams (see :meth:`run_layers`).  chains: with the "tc" engine, runs of consecutive same-shaped layers can go
        through ``bitserial_conv2d_tc_chain`` (one launch per run) where the library accepts them: True = always,
        False = never, "auto" = each such run is timed both ways at set-up and the faster form is kept (the chain wins
        where launches dominate -- small batches -- and loses where every layer already fills the GPU)."""
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
        self.units = self._plan_units(bool(chains) and engine == "tc")
        torch.cuda.synchronize(self.device)   # chained layers fetch filters, scale and bias ahead of stream order
        if chains == "auto":
            self.units = self._keep_faster_units(self.units)
        self.concurrent = concurrent
        self.side = torch.cuda.Stream(device=self.device)
        self.graph = None
        self.static_in = None
        self.launches_per_forward = 2 + len(self.units)

    def _layer_params(self, item):
        """``bs_conv_params`` of a layer as a chain would run it, or None when its output is a slice of a wider tensor."""
        net, L = self.net, item["spec"]
        if L.dst_c_offset != 0 or self.shapes[L.dst][0] != L.O or (L.res and self.shapes[L.res][0] != L.O):
            return None
        return api.conv_params(
            self.bufs[L.src].shape, item["w"].shape, C=L.C, stride=L.stride, pad=L.pad, a_sign=api.UNSIGNED, w_sign=item["w_sign"],
            scale=item["scale"], bias=item["bias"], relu=L.relu, out_bits=net.a_bits, out_sign=api.UNSIGNED,
            residual=self.bufs[L.res] if L.res else None, res_scale=L.res_scale, res_bits=net.a_bits if L.res else 0,
            res_sign=api.UNSIGNED)

    def _plan_units(self, chains: bool) -> List[Dict]:
        """The launches of a forward pass: single layers, and runs of up to MAX_CHAIN consecutive layers that the library
        accepts as one chain (same shape, resident-filter plan) and whose inputs come from outside the run or from an
        earlier layer of it.  Longest run first, greedily from the front."""
        units, i, n = [], 0, len(self.layers)
        while i < n:
            took = 0
            if chains:
                for length in range(min(self.MAX_CHAIN, n - i), 1, -1):
                    items = self.layers[i:i + length]
                    if any(it["w_tc"] is None for it in items):
                        continue
                    prm = [self._layer_params(it) for it in items]
                    if any(q is None for q in prm):
                        continue
                    dsts = [it["spec"].dst for it in items]
                    if len(set(dsts)) != length:
                        continue
                    if any(t in dsts[k:] for k, it in enumerate(items) for t in (it["spec"].src, it["spec"].res) if t):
                        continue
                    nbytes = api.tc_chain_workspace_bytes(prm)
                    if nbytes == 0:
                        continue
                    ws = torch.zeros((nbytes + 3) // 4, dtype=torch.int32, device=self.device)
                    units.append(dict(items=items, params=prm, workspace=ws))
                    took = length
                    break
            if not took:
                units.append(dict(items=[self.layers[i]], params=None, workspace=None))
                took = 1
            i += took
        return units

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

    def _time_units(self, units, reps: int = 8) -> float:
        """Microseconds per pass of `units` launched back to back (as inside a forward pass), from a CUDA graph of `reps` passes."""
        stream = torch.cuda.Stream(device=self.device)
        with torch.cuda.stream(stream):
            for u in units:
                self.run_unit(u, chained=False)
            stream.synchronize()
            graph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(graph, stream=stream):
                for _ in range(reps):
                    for u in units:
                        self.run_unit(u)
            best = float("inf")
            for _ in range(4):
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record(stream)
                graph.replay()
                e1.record(stream)
                e1.synchronize()
                best = min(best, e0.elapsed_time(e1) * 1e3 / reps)
        return best

    def _keep_faster_units(self, units):
        out = []
        for u in units:
            if u["params"] is None:
                out.append(u)
                continue
            singles = [dict(items=[it], params=None, workspace=None) for it in u["items"]]
            t_chain, t_single = self._time_units([u]), self._time_units(singles)
            u["timing_us"] = (t_chain, t_single)
            out.extend([u] if t_chain < t_single else singles)
        torch.cuda.synchronize(self.device)
        return out

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

    def run_unit(self, unit, chained: bool = True) -> None:
        """One launch on the current stream: a layer, or a chain of layers."""
        if unit["params"] is None:
            self.run_layer(unit["items"][0], chained=chained)
            return
        items = unit["items"]
        params = [self._layer_params(it) for it in items]       # pointers of the buffers as they are now (tests swap them)
        api.bitserial_conv2d_tc_chain([self.bufs[it["spec"].src] for it in items], [it["w_tc"] for it in items], params,
                                      [self.bufs[it["spec"].dst] for it in items], unit["workspace"], chained=chained)

    def run_layers(self) -> None:
        """All launches in order.  With ``concurrent`` a single layer whose successor neither reads nor overwrites its
        output (a projection shortcut beside the first conv of its block, the two 1x1 branches of a cross-stage block) is
        launched on a side stream, so the two kernels share the GPU; events carry the dependencies, and under stream
        capture they become the edges of the graph."""
        main = torch.cuda.current_stream(self.device)
        pending: Dict[str, torch.cuda.Event] = {}
        n = len(self.units)

        def touched(unit):
            reads, writes = set(), set()
            for it in unit["items"]:
                L = it["spec"]
                reads.update(t for t in (L.src, L.res) if t)
                writes.add((L.dst, L.dst_c_offset))
            return reads, writes

        for i, unit in enumerate(self.units):
            reads, writes = touched(unit)
            wnames = {d for d, _ in writes}
            aside = False
            if self.concurrent and i + 1 < n and len(unit["items"]) == 1:
                nreads, nwrites = touched(self.units[i + 1])
                aside = (not (wnames & nreads) and not ({d for d, _ in nwrites} & reads) and not (writes & nwrites)
                         and not (reads & set(pending)))
            if aside:
                fork = torch.cuda.Event()
                fork.record(main)
                self.side.wait_event(fork)
                with torch.cuda.stream(self.side):
                    self.run_unit(unit, chained=False)
                    done = torch.cuda.Event()
                    done.record(self.side)
                for d in wnames:
                    pending[d] = done
                continue
            for t in reads | wnames:
                if t in pending:
                    main.wait_event(pending.pop(t))
            self.run_unit(unit)
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
