#!/usr/bin/env python
"""Benchmark of the bit-serial convolution hot path.

One step = one pass of the whole path over one batch: quantise + bitplane-pack the fp32 input, then every
quantised conv layer of the residual stack (conv2_x..conv5_x of an 18-layer network at 224 px, batch 64 per
GPU, 2-bit weights and activations) with the fused requantisation epilogue.  Prints ONE JSON line.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--workload NAME]

`--workload bitwidth_sweep` / `gemm_sweep` time the single-layer sweeps (plane pairs W*A on a 3x3 conv; the im2col-form
matrix products) case by case instead of a layer stack.

N > 1 runs under torchrun, one rank per GPU, each rank its own batch (no data-path collective).
`--impl reference` times the CPU oracle on a bounded sample of the same workload on the host cores.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2207_08820_b200 import workloads as wl  # noqa: E402

ACT_SCALE = 0.25
METRIC = "bitserial_conv_effective_gops"
UNIT = "GOPS"
POPC_PER_CLK_PER_SM = 16          # population count throughput per SM per clock (CUDA programming guide, arithmetic table)
POPC_PER_WORDOP = 2.0 / 3.0       # executed by the kernel's 3:2 carry-save adder: three popc32(AND) word operations cost two counts


def make_net(name: str, batch: int, hw: int = 0):
    """hw: side of the first packed tensor (0: the workload's own: 56 / 320 / 56 / 300)."""
    kw = {"hw": hw} if hw else {}
    if name == "resnet18_body":
        return wl.resnet18_body(batch, **kw), 3000
    if name == "detection_backbone":
        return wl.detection_backbone(batch, **kw), 4000
    if name == "resnet50_body":
        return wl.resnet50_body(batch, **kw), 6000
    if name == "vgg16_ssd_body":
        return wl.vgg16_ssd_body(batch, **kw), 7000
    raise SystemExit(f"unknown workload {name}")


def wordops_per_image(net) -> int:
    """popc32(AND) word operations of the Section V plane-pair sum: outputs x reduction words x plane pairs."""
    shapes = net.tensor_shapes()
    total = 0
    for L in net.layers:
        _, P, Q = shapes[L.dst]
        total += P * Q * L.O * L.k * L.k * ((L.C + 31) // 32) * net.a_bits * net.w_bits
    return total


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            d = json.load(f)
        return d, "measured"
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "sm_max_mhz": 1965.0}, "fallback"


class ClockSampler:
    """Streams nvidia-smi clocks and throttle reasons (one line every 20 ms) while the timed region runs."""
    QUERY = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
             "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.proc = None
        self.lines = []

    def __enter__(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.QUERY}", "--format=csv,noheader,nounits",
                                          "-i", str(self.index), "-lms", "20"], stdout=subprocess.PIPE, text=True)
            time.sleep(0.15)      # let the first samples arrive before the timed region starts
        except Exception:
            self.proc = None
        return self

    def __exit__(self, *exc):
        if self.proc is not None:
            time.sleep(0.05)
            self.proc.terminate()
            try:
                out, _ = self.proc.communicate(timeout=5)
                self.lines = out.splitlines()
            except Exception:
                self.proc.kill()

    def summary(self):
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in self.lines:
            s = [c.strip() for c in line.split(",")]
            try:
                sm.append(float(s[0]))
                mx.append(float(s[1]))
            except (ValueError, IndexError):
                continue
            for n, v in zip(names, s[2:6]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": sorted(reasons), "samples": len(sm)}


def run_reference(args):
    """The CPU oracle, as it stands, on a bounded sample of the workload (host cores only)."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import oracle
    from oracle import network as onet
    net, seed = make_net(args.workload, args.batch, args.hw)
    params = wl.network_params(net, seed)
    sample = args.ref_images
    x = wl.network_input(net, seed, ACT_SCALE, batch=sample)
    macs = net.macs_per_image() * sample
    for _ in range(args.warmup):
        onet.run_stack(net, params, x[:1], ACT_SCALE)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        onet.run_stack(net, params, x, ACT_SCALE)
    dt = (time.perf_counter() - t0) / args.steps
    gops = 2.0 * macs / dt / 1e9
    cores = oracle.num_threads()
    desc = f"{sample} of {net.batch} images of {net.name} per step, all layers, quantise + direct integer conv + epilogue"
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": gops, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": dt * 1e3, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "int32", "data": "synthetic",
        "config": {"workload": f"{net.name}_batch{net.batch}_w{net.w_bits}a{net.a_bits}", "sample_images": sample},
        "images_per_s": sample / dt,
        "cpu_baseline": {"value": gops, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": desc},
        "e2e": {"value": gops, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


def run_sweep(args):
    """Single-layer sweeps on one GPU, one JSON line with a table in "sweep":
      bitwidth_sweep : 3x3 conv N=32, C=O=256, 28x28 for (W,A) in {(1,1),(1,2),(2,2),(2,3),(3,3)}, int32 accumulators +
                       requantised output: time against the number of plane pairs W*A;
      gemm_sweep     : bitserial_gemm, 1-bit bipolar weights x 2-bit activations, M=N in {256,1024,4096}, K in
                       {576,2304,4608}, int32 outputs.
    Every case is launched alone (CUDA events around each launch, L2 flushed before it) on the popcount kernels, the
    conv cases on the tensor-core entry point as well."""
    import torch

    from paper_2207_08820_b200 import api
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the library has no CPU fallback")
    if int(os.environ.get("RANK", "0")) != 0:
        return
    torch.cuda.set_device(0)
    dev = lambda a: torch.from_numpy(np.ascontiguousarray(a)).cuda()
    flush = torch.empty(256 * 1024 * 1024, dtype=torch.uint8, device="cuda")
    flush_words = flush.view(torch.int32)
    peaks, peak_kind = measured_peaks()
    sms = torch.cuda.get_device_properties(0).multi_processor_count
    popc_peak = POPC_PER_CLK_PER_SM * sms * peaks["sm_max_mhz"] * 1e6
    int8_peak = 2.0 * peaks.get("bf16_tflops_sustained", peaks["bf16_tflops"]) * 1e12
    hbm_peak = peaks["hbm_gbs"] * 1e9
    steps = min(args.steps, 20)
    launches = 0

    def timed(fn):
        nonlocal launches
        ts = []
        for k in range(args.warmup + steps):
            flush.zero_()
            torch.amax(flush_words)
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            fn()
            e1.record()
            e1.synchronize()
            if k >= args.warmup:
                ts.append(e0.elapsed_time(e1))
                launches += 1
        return float(np.mean(ts)), float(np.min(ts))

    rows, tot_ops, tot_ms = [], 0.0, 0.0
    with ClockSampler(0) as clocks:
        if args.workload == "bitwidth_sweep":
            for wb, ab in wl.BITWIDTH_SWEEP:
                c = wl.bitwidth_sweep_case(wb, ab)
                xp = api.bitpack_activations(dev(c["x"]), 1.0, ab, c["a_sign"], api.NCHW)
                wp = api.pack_weights(dev(c["w"]), wb, c["w_sign"])
                sc, bi = dev(c["scale"]), dev(c["bias"])
                P = Q = c["H"]
                acc = torch.empty(c["N"], c["O"], P, Q, dtype=torch.int32, device="cuda")
                outp = torch.zeros(c["N"], P, Q, c["O"] // 32, ab, dtype=torch.int32, device="cuda")
                kw = dict(C=c["C"], stride=1, pad=1, a_sign=c["a_sign"], w_sign=c["w_sign"], scale=sc, bias=bi, relu=True,
                          out_bits=ab, out_sign=api.UNSIGNED, out_packed=outp)
                macs = c["N"] * P * Q * c["O"] * c["C"] * 9
                wops = macs // 32 * wb * ab
                ms_acc, _ = timed(lambda: api.bitserial_conv2d(xp, wp, out_i32=acc, **kw))     # int32 + packed outputs
                ms, best = timed(lambda: api.bitserial_conv2d(xp, wp, **kw))                   # packed output only
                row = {"w_bits": wb, "a_bits": ab, "pairs": wb * ab, "ms": ms, "ms_best": best, "ms_with_int32_out": ms_acc,
                       "gops": 2.0 * macs / ms / 1e6, "Tword_ops_per_s": wops / ms / 1e9, "frac_popc": wops / (ms * 1e-3) / popc_peak}
                if api.tc_supported(c["N"], c["C"], c["H"], c["W"], c["O"], 3, 1, 1, ab, c["a_sign"], wb, c["w_sign"]):
                    wt = api.tc_prepare_weights(wp, c["C"], c["w_sign"], ab)
                    tms, _ = timed(lambda: api.bitserial_conv2d(xp, wp, wgt_tc=wt, **kw))
                    row.update(tc_ms=tms, tc_gops=2.0 * macs / tms / 1e6, tc_frac_int8=2.0 * macs / (tms * 1e-3) / int8_peak)
                rows.append(row)
                tot_ops += 2.0 * macs
                tot_ms += ms
            name = "bitwidth_sweep_conv3x3_n32_c256_o256_hw28"
        else:
            for M in wl.GEMM_SWEEP_MN:
                for K in wl.GEMM_SWEEP_K:
                    c = wl.gemm_case(M, M, K, seed=wl.gemm_sweep_seed(M, K))
                    a_p = api.bs_pack_rows(dev(c["a"]), c["a_bits"], c["a_sign"])
                    w_p = api.bs_pack_rows(dev(c["w"]), c["w_bits"], c["w_sign"])
                    out = torch.empty(M, M, dtype=torch.int32, device="cuda")
                    ms, best = timed(lambda: api.bitserial_gemm(a_p, w_p, K, a_sign=c["a_sign"], w_sign=c["w_sign"], out_i32=out))
                    macs = M * M * K
                    wops = macs // 32 * c["a_bits"] * c["w_bits"]
                    nbytes = (a_p.numel() + w_p.numel() + out.numel()) * 4
                    t_popc, t_hbm = wops / popc_peak, nbytes / hbm_peak
                    row = {"M": M, "N": M, "K": K, "ms": ms, "ms_best": best, "gops": 2.0 * macs / ms / 1e6,
                           "Tword_ops_per_s": wops / ms / 1e9, "GB_per_s": nbytes / ms / 1e6,
                           "bound": "alu" if t_popc >= t_hbm else "hbm",
                           "frac_roofline": max(t_popc, t_hbm) / (ms * 1e-3)}
                    # the same product on the tensor-core entry point: bound by the int8 rate or by the int32 output
                    wt = api.tc_prepare_weights(w_p.view(M, 1, 1, -1, c["w_bits"]), K, c["w_sign"], c["a_bits"])
                    tms, _ = timed(lambda: api.bitserial_gemm_tc(a_p, wt, M, K, c["w_bits"], a_sign=c["a_sign"], w_sign=c["w_sign"]))
                    t_tc, t_hbm_tc = 2.0 * macs / int8_peak, (a_p.numel() * 4 + wt.numel() + out.numel() * 4) / hbm_peak
                    row.update(tc_ms=tms, tc_gops=2.0 * macs / tms / 1e6, tc_bound="tensor" if t_tc >= t_hbm_tc else "hbm",
                               tc_frac_roofline=max(t_tc, t_hbm_tc) / (tms * 1e-3))
                    rows.append(row)
                    tot_ops += 2.0 * macs
                    tot_ms += ms
            name = "gemm_sweep_w1bipolar_a2_int32_out"
    api.bs_check_status()
    print(json.dumps({
        "metric": METRIC, "value": tot_ops / tot_ms / 1e6, "unit": UNIT, "n_gpus": 1, "steps": steps, "warmup": args.warmup,
        "ms_per_step": tot_ms, "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "int32",
        "data": "synthetic",
        "config": {"workload": name, "engine": "popc", "l2": "flushed before every launch (256 MB write, then read back)",
                   "launch": "one eager launch per case, CUDA events around it (launch latency included)"},
        "sweep": rows,
        "peaks": {"popc_word_ops_per_s": popc_peak, "int8_ops_per_s": int8_peak, "hbm_bytes_per_s": hbm_peak, "kind": peak_kind},
        "gpu_launches": launches, "clocks": clocks.summary()}))


def run_ours(args):
    import torch
    import torch.distributed as dist

    from paper_2207_08820_b200 import api, replicas
    from paper_2207_08820_b200.net import BitserialNet

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the library has no CPU fallback")
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))

    net, seed = make_net(args.workload, args.batch, args.hw)
    params = wl.network_params(net, seed)
    x_host = torch.from_numpy(wl.network_input(net, replicas.rank_seed(seed, rank), ACT_SCALE)).pin_memory()
    x_dev = x_host.cuda()
    runner = BitserialNet(net, params, ACT_SCALE, batch=net.batch, engine=args.engine)

    stream = torch.cuda.Stream()
    with torch.cuda.stream(stream):
        # two graphs so that the pack kernel and the conv kernels can be timed separately on this stream
        in_buf = runner.bufs[net.in_name]
        api.bitpack_activations(x_dev, ACT_SCALE, net.a_bits, api.UNSIGNED, api.NCHW, out=in_buf.view(-1))
        runner.forward(x_dev)
        api.bs_check_status(stream)
        def run_pack():
            runner.pack_input(x_dev)

        def run_convs():
            runner.run_layers()

        if args.eager:
            replay_pack, replay_conv = run_pack, run_convs
        else:
            g_pack, g_conv = torch.cuda.CUDAGraph(), torch.cuda.CUDAGraph()
            with torch.cuda.graph(g_pack, stream=stream):
                run_pack()
            with torch.cuda.graph(g_conv, stream=stream):
                run_convs()
            replay_pack, replay_conv = g_pack.replay, g_conv.replay
    stream.synchronize()

    flush = torch.empty(256 * 1024 * 1024, dtype=torch.uint8, device="cuda")   # larger than the 126 MB L2
    flush_words = flush.view(torch.int32)

    def flush_l2():
        """Write a buffer larger than L2, then read it back: the write evicts every line of the step, the read
        drains the dirty lines the write left, so the timed kernels start on a cold AND clean L2 instead of paying
        for the flush's write-backs."""
        flush.zero_()
        torch.amax(flush_words)

    def step(ev=None):
        if ev:
            ev[0].record(stream)
        replay_pack()
        if ev:
            ev[1].record(stream)
        replay_conv()
        if ev:
            ev[2].record(stream)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    out_packed = runner.bufs[net.out_name]
    out_host = torch.empty(out_packed.shape, dtype=out_packed.dtype).pin_memory()

    with torch.cuda.stream(stream):
        for _ in range(args.warmup):
            flush_l2()
            step()
        barrier()
        events = [[torch.cuda.Event(enable_timing=True) for _ in range(3)] for _ in range(args.steps)]
        with ClockSampler(local) as clocks:
            barrier()
            for k in range(args.steps):
                flush_l2()             # L2 flush between timed iterations (outside the event pairs)
                step(events[k])
            barrier()
        t_pack = sum(e[0].elapsed_time(e[1]) for e in events) / args.steps
        t_conv = sum(e[1].elapsed_time(e[2]) for e in events) / args.steps
        t_step = sum(e[0].elapsed_time(e[2]) for e in events) / args.steps
        api.bs_check_status(stream)

        # end to end through the public API: pinned host input -> device, path, packed result -> host, every step.
        # Two device input buffers: the host -> device copy of step k+1 (copy stream) runs beside the kernels of step
        # k (compute stream), the device -> host read of the result on a third stream; the L2 flush stays inside the
        # timed region on the compute stream.  Timed with CUDA events on the compute stream around all steps.
        x_dev_b = [x_dev, torch.empty_like(x_dev)]
        if args.eager:
            packs = [run_pack, None]
        else:
            g_pack_b = torch.cuda.CUDAGraph()
            def run_pack_b():
                runner.pack_input(x_dev_b[1])
            run_pack_b()
            stream.synchronize()
            with torch.cuda.graph(g_pack_b, stream=stream):
                run_pack_b()
            packs = [replay_pack, g_pack_b.replay]
        h2d_stream, d2h_stream = torch.cuda.Stream(), torch.cuda.Stream()
        ev_h2d = [torch.cuda.Event() for _ in range(2)]
        ev_read = [torch.cuda.Event() for _ in range(2)]       # the pack kernel has consumed input buffer b
        ev_out, ev_d2h = torch.cuda.Event(), torch.cuda.Event()
        e2e_ev = [torch.cuda.Event(enable_timing=True) for _ in range(2)]
        for b_ in range(2):
            ev_read[b_].record(stream)
        ev_d2h.record(stream)
        stream.synchronize()
        for k in range(args.warmup + args.steps):
            bi = k % 2 if packs[1] is not None else 0
            if k == args.warmup:
                stream.wait_event(ev_d2h)                      # the warm-up steps have drained
                e2e_ev[0].record(stream)
                h2d_stream.wait_event(e2e_ev[0])               # no timed copy starts before the start mark
            h2d_stream.wait_event(ev_read[bi])
            with torch.cuda.stream(h2d_stream):
                x_dev_b[bi].copy_(x_host, non_blocking=True)
                ev_h2d[bi].record(h2d_stream)
            flush.zero_()
            stream.wait_event(ev_h2d[bi])
            packs[bi]()
            ev_read[bi].record(stream)
            stream.wait_event(ev_d2h)                          # the previous result has left the output buffer
            replay_conv()
            ev_out.record(stream)
            d2h_stream.wait_event(ev_out)
            with torch.cuda.stream(d2h_stream):
                out_host.copy_(out_packed, non_blocking=True)
                ev_d2h.record(d2h_stream)
        stream.wait_event(ev_d2h)
        e2e_ev[1].record(stream)
        barrier()
        t_e2e = e2e_ev[0].elapsed_time(e2e_ev[1]) / args.steps

        # the other engine on the same inputs, conv layers only (reported beside the headline, not part of it)
        other = "popc" if args.engine == "tc" else "tc"
        t_conv_other = None
        if world == 1 and not args.eager:
            runner2 = BitserialNet(net, params, ACT_SCALE, batch=net.batch, engine=other)
            runner2.bufs[net.in_name].copy_(in_buf)
            runner2.run_layers()
            stream.synchronize()
            g2 = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g2, stream=stream):
                runner2.run_layers()
            n2 = min(args.steps, 10)
            ev2 = [[torch.cuda.Event(enable_timing=True) for _ in range(2)] for _ in range(n2)]
            for k in range(3 + n2):
                flush_l2()
                if k >= 3:
                    ev2[k - 3][0].record(stream)
                g2.replay()
                if k >= 3:
                    ev2[k - 3][1].record(stream)
            stream.synchronize()
            api.bs_check_status(stream)
            t_conv_other = sum(e[0].elapsed_time(e[1]) for e in ev2) / n2

    t_step, t_e2e, t_conv, t_pack = replicas.max_over_ranks([t_step, t_e2e, t_conv, t_pack], torch.device("cuda", local))

    if rank == 0:
        macs = net.macs_per_image() * net.batch
        wops = wordops_per_image(net) * net.batch
        gops = 2.0 * macs * world / (t_step * 1e-3) / 1e9
        peaks, peak_kind = measured_peaks()
        sms = torch.cuda.get_device_properties(local).multi_processor_count
        popc_peak = POPC_PER_CLK_PER_SM * sms * peaks["sm_max_mhz"] * 1e6          # counts/s at the maximum SM clock
        popc_measured = api.bs_popc_rate(4096)
        int8_peak_tops = 2.0 * peaks.get("bf16_tflops_sustained", peaks["bf16_tflops"])   # dense int8 = 2 x bf16 (nominal ratio)

        def popc_roofline(t_ms):
            a = wops / (t_ms * 1e-3)
            return {"bound": "alu", "kernel": "bitserial_conv_kernel", "achieved": a / 1e12, "peak": popc_peak / 1e12,
                    "unit": "Tword-op/s", "frac": a / popc_peak, "traffic": None,
                    "peak_source": f"{POPC_PER_CLK_PER_SM} popc/clk/SM x {sms} SMs x {peaks['sm_max_mhz']:.0f} MHz ({peak_kind} clock); "
                                   "achieved counts ALGORITHMIC word operations, the kernel's 3:2 carry-save adder executes 2/3 "
                                   "as many population counts, so frac can exceed 1 (frac_executed is on the executed counts)",
                    "frac_executed": a * POPC_PER_WORDOP / popc_peak,
                    "popc_pipe_measured": popc_measured / 1e12, "launches_per_step": len(net.layers),
                    "avg_launch_ms": t_ms / len(net.layers)}

        # dram__bytes_read + dram__bytes_write per launch (mean of the 19 launches of one pass) from the ncu capture of
        # these kernels on this workload; other workloads have no capture
        tc_traffic = 57.53e6 / 19 if (net.name == "resnet18_body" and net.batch == 64) else None

        def tensor_roofline(t_ms):
            a = 2.0 * macs / (t_ms * 1e-3) / 1e12
            return {"bound": "tensor", "kernel": "bitserial_conv_tc_persistent_kernel", "achieved": a, "peak": int8_peak_tops,
                    "unit": "TOP/s", "frac": a / int8_peak_tops, "traffic": tc_traffic,
                    "peak_source": f"2 x {peak_kind} sustained bf16 cuBLAS TFLOP/s (nominal int8:bf16 ratio)",
                    "launches_per_step": len(net.layers), "avg_launch_ms": t_ms / len(net.layers)}

        roof = tensor_roofline(t_conv) if args.engine == "tc" else popc_roofline(t_conv)
        in_bytes = x_host.numel() * 4
        pack_bytes = in_bytes + in_buf.numel() * 4
        line = {
            "metric": METRIC, "value": gops, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": t_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "int32", "data": "synthetic",
            "config": {"workload": f"{net.name}_batch{net.batch}_w{net.w_bits}a{net.a_bits}" + (f"_hw{args.hw}" if args.hw else ""),
                       "global_batch": net.batch * world, "parallelism": f"replicas{world}", "layers": len(net.layers),
                       "l2": "flushed between timed iterations (256 MB write, then read back so no dirty lines are left)", "launch": ("eager stream launches" if args.eager else "CUDA graphs (pack, convs)") +
                                 "; layers chained (programmatic dependent launch), independent neighbours on two streams"},
            "images_per_s": net.batch * world / (t_step * 1e-3),
            "roofline": roof,
            "pack": {"bound": "hbm", "ms": t_pack, "achieved": pack_bytes / (t_pack * 1e-3) / 1e9, "peak": peaks["hbm_gbs"],
                     "unit": "GB/s", "frac": pack_bytes / (t_pack * 1e-3) / 1e9 / peaks["hbm_gbs"]},
            "e2e": {"value": 2.0 * macs * world / (t_e2e * 1e-3) / 1e9, "unit": UNIT, "ms_per_step": t_e2e, "overlap": "h2d of step k+1 beside the kernels of step k (two input buffers); L2 flush inside",
                    "h2d_bytes_per_step": in_bytes, "d2h_bytes_per_step": out_host.numel() * 4},
            "gpu_launches": runner.launches_per_forward * args.steps,
            "clocks": clocks.summary(),
        }
        line["config"]["engine"] = args.engine
        if t_conv_other is not None:
            alt = popc_roofline(t_conv_other) if other == "popc" else tensor_roofline(t_conv_other)
            alt["engine"] = other
            alt["conv_ms"] = t_conv_other
            line["other_engine"] = alt
        if world == 1 and not args.no_cpu_baseline:
            line["cpu_baseline"] = cpu_baseline(net, params, seed, args.cpu_baseline_images)
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


def cpu_baseline(net, params, seed, sample):
    import oracle
    from oracle import network as onet
    x = wl.network_input(net, seed, ACT_SCALE, batch=sample)
    onet.run_stack(net, params, x[:1], ACT_SCALE)
    t0 = time.perf_counter()
    onet.run_stack(net, params, x, ACT_SCALE)
    dt = time.perf_counter() - t0
    return {"value": 2.0 * net.macs_per_image() * sample / dt / 1e9, "unit": UNIT, "cores": oracle.num_threads(),
            "kind": "oracle", "images_per_s": sample / dt,
            "sample": f"{sample} of {net.batch} images of {net.name}, all layers, one pass ({dt:.1f} s)"}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=50)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="resnet18_body", choices=["resnet18_body", "detection_backbone", "resnet50_body", "vgg16_ssd_body", "bitwidth_sweep", "gemm_sweep"])
    ap.add_argument("--hw", type=int, default=0, help="side of the first packed tensor (default: the workload's own; the paper's 320 / 352 px "
                    "detection inputs are --workload detection_backbone --hw 160 / 176)")
    ap.add_argument("--batch", type=int, default=0, help="images per GPU (default: 64 / 16 / 32 / 8 as the workload defines)")
    ap.add_argument("--ref-images", type=int, default=2, help="images per step of the reference arm (bounded CPU sample)")
    ap.add_argument("--cpu-baseline-images", type=int, default=64, help="images of the one oracle pass timed beside the GPU run")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--engine", default="tc", choices=["popc", "tc"],
                    help="popc: popcount kernels on the integer pipes; tc: exact int8 tensor-core formulation")
    ap.add_argument("--eager", action="store_true", help="plain stream launches instead of CUDA graphs (for per-launch profiling)")
    args = ap.parse_args()
    if args.workload in ("bitwidth_sweep", "gemm_sweep"):
        if args.impl == "reference":
            raise SystemExit("the reference arm times the layer stacks only")
        args.warmup = max(args.warmup, 3)
        return run_sweep(args)
    if args.batch == 0:
        args.batch = {"resnet18_body": 64, "detection_backbone": 16, "resnet50_body": 32, "vgg16_ssd_body": 8}[args.workload]
    if args.warmup < 3 and args.impl == "ours":
        args.warmup = 3
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
