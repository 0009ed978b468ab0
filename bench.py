#!/usr/bin/env python
"""Benchmark of the bit-serial convolution hot path.

One step = one pass of the whole path over one batch: quantise + bitplane-pack the fp32 input, then every
quantised conv layer of the residual stack (conv2_x..conv5_x of an 18-layer network at 224 px, batch 64 per
GPU, 2-bit weights and activations) with the fused requantisation epilogue.  Prints ONE JSON line.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--workload NAME]

`--workload bitwidth_sweep` / `gemm_sweep` time the single-layer sweeps (plane pairs W*A on a 3x3 conv; the im2col-form
matrix products) case by case instead of a layer stack.

The default line also carries, under "configs", compact measurements of the other workloads the metric is defined on
(the single 3x3 layer with its launch floor, the matrix-product sweep, the detection-shaped stack, the bit-width sweep)
and, under "pack_large", the pack kernels on inputs larger than the L2 cache; `--no-configs` leaves them out.

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


def layer_roofline(net, engine: str, peaks: dict, popc_peak: float):
    """Per layer: algorithmic work, minimum bytes, and the roofline time max(t_compute, t_hbm) on both tensor denominators.
    Returns (rows, sums).  Minimum bytes of a layer: packed input once + filters (int8 tiles on the tensor-core engine, packed
    planes on the popcount engine) + residual + packed output."""
    shapes = net.tensor_shapes()
    hbm = peaks["hbm_gbs"] * 1e9
    int8_burst = 2.0 * peaks["bf16_tflops"] * 1e12
    int8_sust = 2.0 * peaks.get("bf16_tflops_sustained", peaks["bf16_tflops"]) * 1e12
    rows = []
    for L in net.layers:
        Cs, H, W = shapes[L.src]
        Cd, P, Q = shapes[L.dst]
        macs = net.batch * P * Q * L.O * L.C * L.k * L.k
        wops = macs // 32 * net.a_bits * net.w_bits if L.C % 32 == 0 else net.batch * P * Q * L.O * L.k * L.k * ((L.C + 31) // 32) * net.a_bits * net.w_bits
        act_bytes = net.batch * H * W * ((L.C + 31) // 32) * net.a_bits * 4
        wgt_bytes = (((L.O + 127) // 128) * 128 * L.k * L.k * L.C) if engine == "tc" else L.O * L.k * L.k * ((L.C + 31) // 32) * net.w_bits * 4
        out_bytes = net.batch * P * Q * ((L.O + 31) // 32) * net.a_bits * 4
        res_bytes = out_bytes if L.res else 0
        nbytes = act_bytes + wgt_bytes + out_bytes + res_bytes
        t_hbm = nbytes / hbm
        if engine == "tc":
            tb, ts = 2.0 * macs / int8_burst, 2.0 * macs / int8_sust
        else:
            tb = ts = wops / popc_peak
        rows.append({"name": L.name, "macs": macs, "wordops": wops, "bytes": nbytes, "t_hbm": t_hbm, "t_compute_burst": tb,
                     "t_compute_sustained": ts, "bound": "hbm" if t_hbm > tb else ("tensor" if engine == "tc" else "alu")})
    sums = {"roofline_s_burst": sum(max(r["t_hbm"], r["t_compute_burst"]) for r in rows),
            "roofline_s_sustained": sum(max(r["t_hbm"], r["t_compute_sustained"]) for r in rows),
            "bytes": sum(r["bytes"] for r in rows), "hbm_bound_layers": sum(r["bound"] == "hbm" for r in rows)}
    return rows, sums


def captured_traffic(net_name: str, batch: int):
    """dram__bytes_read + dram__bytes_write of one pass of the conv launches, from the tracked ncu summary of that capture
    under profiles/.  The summary names the SHA-256 of the kernel source it was taken on; a different source gives None
    (the counters are stale once the kernel has changed)."""
    import hashlib
    import re
    path = os.path.join(ROOT, "profiles", f"bitserial_conv_tc_kernels_{net_name}_dram_traffic.md")
    src = os.path.join(ROOT, "paper_2207_08820_b200", "csrc", "tc_conv.cu")
    if not (os.path.exists(path) and os.path.exists(src)):
        return None, None
    text = open(path).read()
    m_bytes = re.search(r"traffic_bytes_per_pass:\s*([0-9.eE+]+)", text)
    m_batch = re.search(r"batch:\s*(\d+)", text)
    m_sha = re.search(r"kernel_source_sha256:\s*([0-9a-f]{64})", text)
    if not (m_bytes and m_sha and m_batch) or int(m_batch.group(1)) != batch:
        return None, os.path.basename(path)
    if hashlib.sha256(open(src, "rb").read()).hexdigest() != m_sha.group(1):
        return None, os.path.basename(path) + " (stale: the kernel source changed after the capture)"
    return float(m_bytes.group(1)), os.path.basename(path)


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


class LaunchTimer:
    """Times single launches: L2 flushed (256 MB write, then read back) before each, CUDA events around it."""

    def __init__(self, torch, warmup: int, steps: int):
        self.torch = torch
        self.warmup, self.steps = warmup, steps
        self.flush = torch.empty(256 * 1024 * 1024, dtype=torch.uint8, device="cuda")
        self.flush_words = self.flush.view(torch.int32)
        self.launches = 0

    def __call__(self, fn):
        torch = self.torch
        ts = []
        for k in range(self.warmup + self.steps):
            self.flush.zero_()
            torch.amax(self.flush_words)
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            fn()
            e1.record()
            e1.synchronize()
            if k >= self.warmup:
                ts.append(e0.elapsed_time(e1))
                self.launches += 1
        return float(np.mean(ts)), float(np.min(ts))


def sweep_peaks(torch):
    peaks, peak_kind = measured_peaks()
    sms = torch.cuda.get_device_properties(0).multi_processor_count
    return {"popc": POPC_PER_CLK_PER_SM * sms * peaks["sm_max_mhz"] * 1e6, "int8_burst": 2.0 * peaks["bf16_tflops"] * 1e12,
            "int8_sustained": 2.0 * peaks.get("bf16_tflops_sustained", peaks["bf16_tflops"]) * 1e12,
            "hbm": peaks["hbm_gbs"] * 1e9, "kind": peak_kind}


def measure_bitwidth_sweep(torch, api, timed, pk):
    """3x3 conv N=32, C=O=256, 28x28 for (W,A) in {(1,1),(1,2),(2,2),(2,3),(3,3)}: time against the plane pairs W*A."""
    dev = lambda a: torch.from_numpy(np.ascontiguousarray(a)).cuda()
    rows, tot_ops, tot_ms = [], 0.0, 0.0
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
               "gops": 2.0 * macs / ms / 1e6, "Tword_ops_per_s": wops / ms / 1e9,
               "frac_popc_algorithmic": wops / (ms * 1e-3) / pk["popc"],
               "frac_popc_executed": wops * POPC_PER_WORDOP / (ms * 1e-3) / pk["popc"]}
        if api.tc_supported(c["N"], c["C"], c["H"], c["W"], c["O"], 3, 1, 1, ab, c["a_sign"], wb, c["w_sign"]):
            wt = api.tc_prepare_weights(wp, c["C"], c["w_sign"], ab)
            tms, _ = timed(lambda: api.bitserial_conv2d(xp, wp, wgt_tc=wt, **kw))
            row.update(tc_ms=tms, tc_gops=2.0 * macs / tms / 1e6, tc_frac_int8_burst=2.0 * macs / (tms * 1e-3) / pk["int8_burst"],
                       tc_frac_int8_sustained=2.0 * macs / (tms * 1e-3) / pk["int8_sustained"])
        rows.append(row)
        tot_ops += 2.0 * macs
        tot_ms += ms
    return rows, tot_ops, tot_ms


def measure_gemm_sweep(torch, api, timed, pk):
    """bitserial_gemm and bitserial_gemm_tc, 1-bit bipolar weights x 2-bit activations, M=N in {256,1024,4096}, K in
    {576,2304,4608}, int32 outputs; per shape the binding roofline (integer pipe / tensor core or the int32 output traffic)."""
    dev = lambda a: torch.from_numpy(np.ascontiguousarray(a)).cuda()
    rows, tot_ops, tot_ms = [], 0.0, 0.0
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
            t_popc, t_hbm = wops * POPC_PER_WORDOP / pk["popc"], nbytes / pk["hbm"]       # executed counts (3:2 carry-save adder)
            row = {"M": M, "N": M, "K": K, "ms": ms, "ms_best": best, "gops": 2.0 * macs / ms / 1e6,
                   "Tword_ops_per_s": wops / ms / 1e9, "GB_per_s": nbytes / ms / 1e6,
                   "bound": "alu" if t_popc >= t_hbm else "hbm", "frac": max(t_popc, t_hbm) / (ms * 1e-3),
                   "frac_algorithmic": max(wops / pk["popc"], t_hbm) / (ms * 1e-3)}
            wt = api.tc_prepare_weights(w_p.view(M, 1, 1, -1, c["w_bits"]), K, c["w_sign"], c["a_bits"])
            tms, _ = timed(lambda: api.bitserial_gemm_tc(a_p, wt, M, K, c["w_bits"], a_sign=c["a_sign"], w_sign=c["w_sign"], out_i32=out))
            t_tc, t_hbm_tc = 2.0 * macs / pk["int8_burst"], (a_p.numel() * 4 + wt.numel() + out.numel() * 4) / pk["hbm"]
            row.update(tc_ms=tms, tc_gops=2.0 * macs / tms / 1e6, tc_bound="tensor" if t_tc >= t_hbm_tc else "hbm",
                       tc_frac=max(t_tc, t_hbm_tc) / (tms * 1e-3))
            rows.append(row)
            tot_ops += 2.0 * macs
            tot_ms += ms
    return rows, tot_ops, tot_ms


def run_sweep(args):
    """Single-layer sweeps on one GPU, one JSON line with a table in "sweep" (see measure_bitwidth_sweep / measure_gemm_sweep).
    Every case is launched alone (CUDA events around each launch, L2 flushed before it)."""
    import torch

    from paper_2207_08820_b200 import api
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the library has no CPU fallback")
    if int(os.environ.get("RANK", "0")) != 0:
        return
    torch.cuda.set_device(0)
    pk = sweep_peaks(torch)
    steps = min(args.steps, 20)
    timed = LaunchTimer(torch, args.warmup, steps)
    with ClockSampler(0) as clocks:
        if args.workload == "bitwidth_sweep":
            rows, tot_ops, tot_ms = measure_bitwidth_sweep(torch, api, timed, pk)
            name = "bitwidth_sweep_conv3x3_n32_c256_o256_hw28"
        else:
            rows, tot_ops, tot_ms = measure_gemm_sweep(torch, api, timed, pk)
            name = "gemm_sweep_w1bipolar_a2_int32_out"
    api.bs_check_status()
    print(json.dumps({
        "metric": METRIC, "value": tot_ops / tot_ms / 1e6, "unit": UNIT, "n_gpus": 1, "steps": steps, "warmup": args.warmup,
        "ms_per_step": tot_ms, "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "int32",
        "data": "synthetic",
        "config": {"workload": name, "engine": "popc", "l2": "flushed before every launch (256 MB write, then read back)",
                   "launch": "one eager launch per case, CUDA events around it (launch latency included)"},
        "sweep": rows,
        "peaks": {"popc_word_ops_per_s": pk["popc"], "int8_ops_per_s_burst": pk["int8_burst"], "int8_ops_per_s_sustained": pk["int8_sustained"],
                  "hbm_bytes_per_s": pk["hbm"], "kind": pk["kind"]},
        "gpu_launches": timed.launches, "clocks": clocks.summary()}))


def measure_other_configs(torch, api, stream, args):
    """The workloads besides the headline stack, measured compactly inside the default run (one GPU, rank 0):
      single_layer   3x3 conv 1x64x56x56, 64 filters, W2A2: time per launch on both engines inside a CUDA graph of 20 launches, and
                     the launch floor (a one-tile launch of each engine, same method);
      gemm_sweep / bitwidth_sweep   as the stand-alone sweeps, fewer repetitions;
      detection_backbone            the detection-shaped stack at batch 16 on the tensor-core engine: conv time per pass under a
                                    CUDA graph, images/s, and sum(roofline time) / measured time over its layers;
      layer_chains   the residual stack's conv layers at batch 16 and 64, one launch per layer against runs of same-shaped
                     layers as one launch (bitserial_conv2d_tc_chain), and how many launches the runner's set-up timing keeps;
      pack_large     the pack kernels on inputs larger than L2 (fp32 NCHW and NHWC, 2 and 3 bits)."""
    from paper_2207_08820_b200.net import BitserialNet
    dev = lambda a: torch.from_numpy(np.ascontiguousarray(a)).cuda()
    pk = sweep_peaks(torch)
    peaks, _ = measured_peaks()
    out = {}
    launches = 0

    def graph_time(fn, reps=20, rounds=5):
        nonlocal launches
        with torch.cuda.stream(stream):
            fn()
            stream.synchronize()
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g, stream=stream):
                for _ in range(reps):
                    fn()
            ts = []
            for k in range(rounds + 2):
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record(stream)
                g.replay()
                e1.record(stream)
                e1.synchronize()
                if k >= 2:
                    ts.append(e0.elapsed_time(e1) / reps)
                    launches += reps
        return float(np.mean(ts))

    # ---- the single 3x3 layer and the launch floor
    c = wl.single_conv_case(seed=0, calibrated=True)
    xp = api.bitpack_activations(dev(c["x"]), 1.0, 2, 0, api.NCHW)
    wp = api.pack_weights(dev(c["w"]), 2, c["w_sign"])
    wt = api.tc_prepare_weights(wp, 64, c["w_sign"], 2)
    sc, bi = dev(c["scale"]), dev(c["bias"])
    outp = torch.zeros(1, 56, 56, 2, 2, dtype=torch.int32, device="cuda")
    kw = dict(C=64, stride=1, pad=1, a_sign=0, w_sign=c["w_sign"], scale=sc, bias=bi, relu=True, out_bits=2, out_packed=outp)
    t_popc = graph_time(lambda: api.bitserial_conv2d(xp, wp, **kw))
    t_tc = graph_time(lambda: api.bitserial_conv2d(xp, wp, wgt_tc=wt, **kw))
    tiny = wl.single_conv_case(seed=1, N=1, C=64, H=8, W=8, O=32, k=1, stride=1, pad=0, calibrated=True)
    txp = api.bitpack_activations(dev(tiny["x"]), 1.0, 2, 0, api.NCHW)
    twp = api.pack_weights(dev(tiny["w"]), 2, tiny["w_sign"])
    twt = api.tc_prepare_weights(twp, 64, tiny["w_sign"], 2)
    toutp = torch.zeros(1, 8, 8, 1, 2, dtype=torch.int32, device="cuda")
    tkw = dict(C=64, stride=1, pad=0, a_sign=0, w_sign=tiny["w_sign"], scale=dev(tiny["scale"]), bias=dev(tiny["bias"]), relu=True,
               out_bits=2, out_packed=toutp)
    f_popc = graph_time(lambda: api.bitserial_conv2d(txp, twp, **tkw))
    f_tc = graph_time(lambda: api.bitserial_conv2d(txp, twp, wgt_tc=twt, **tkw))
    macs1 = 56 * 56 * 64 * 64 * 9
    out["single_layer"] = {"workload": "conv3x3_n1_c64_o64_hw56_w2a2 (warm L2, 20 launches per CUDA graph)",
                           "popc_us": t_popc * 1e3, "tc_us": t_tc * 1e3, "popc_gops": 2.0 * macs1 / t_popc / 1e6, "tc_gops": 2.0 * macs1 / t_tc / 1e6,
                           "launch_floor_us": {"popc": f_popc * 1e3, "tc": f_tc * 1e3, "what": "one-tile launch (1x1 conv on an 8x8 image), same method"},
                           "roofline_us": {"popc_executed": macs1 // 32 * 4 * POPC_PER_WORDOP / pk["popc"] * 1e6, "tensor_burst": 2.0 * macs1 / pk["int8_burst"] * 1e6},
                           "bound": "launch latency: the layer's arithmetic is shorter than one launch"}
    # ---- sweeps
    timed = LaunchTimer(torch, 2, 5)
    rows, _, _ = measure_gemm_sweep(torch, api, timed, pk)
    out["gemm_sweep"] = [{k: (round(v, 5) if isinstance(v, float) else v) for k, v in r.items()
                          if k in ("M", "K", "ms", "bound", "frac", "frac_algorithmic", "tc_ms", "tc_bound", "tc_frac")} for r in rows]
    rows, _, _ = measure_bitwidth_sweep(torch, api, timed, pk)
    out["bitwidth_sweep"] = [{k: (round(v, 5) if isinstance(v, float) else v) for k, v in r.items()
                              if k in ("w_bits", "a_bits", "pairs", "ms", "Tword_ops_per_s", "frac_popc_algorithmic", "frac_popc_executed", "tc_ms",
                                       "tc_frac_int8_burst")} for r in rows]
    launches += timed.launches
    # ---- pack kernels on inputs larger than L2
    packs = []
    for layout, shape in ((api.NCHW, (256, 64, 56, 56)), (api.NHWC, (256, 56, 56, 64))):
        x = torch.empty(shape, dtype=torch.float32, device="cuda").uniform_(-0.2, 0.9)
        for bits in (2, 3):
            n = x.numel()
            outw = torch.empty(n // 32 * bits, dtype=torch.int32, device="cuda")
            ms = graph_time(lambda: api.bitpack_activations(x, ACT_SCALE, bits, api.UNSIGNED, layout, out=outw), reps=5, rounds=4)
            nbytes = n * 4 + outw.numel() * 4
            packs.append({"layout": "nchw" if layout == api.NCHW else "nhwc", "bits": bits, "input_MB": n * 4 / 1e6, "ms": ms,
                          "GB_per_s": nbytes / ms / 1e6, "frac_hbm": nbytes / (ms * 1e-3) / pk["hbm"]})
        del x
    out["pack_large"] = packs
    # ---- the detection-shaped stack
    net, seed = make_net("detection_backbone", 16)
    params = wl.network_params(net, seed)
    x = torch.from_numpy(wl.network_input(net, seed, ACT_SCALE)).cuda()
    runner = BitserialNet(net, params, ACT_SCALE, batch=net.batch, engine="tc")
    with torch.cuda.stream(stream):
        runner.forward(x)
        stream.synchronize()
        t_pack = graph_time(lambda: runner.pack_input(x), reps=1, rounds=5)
        t_conv = graph_time(runner.run_layers, reps=1, rounds=8)
    _, sums = layer_roofline(net, "tc", peaks, pk["popc"])
    macs = net.macs_per_image() * net.batch
    launches += 0
    out["detection_backbone"] = {"workload": f"{net.name}_batch{net.batch}_w2a2 (warm L2, one CUDA graph per pass)", "layers": len(net.layers),
                                 "conv_ms": t_conv, "pack_ms": t_pack, "images_per_s": net.batch / ((t_conv + t_pack) * 1e-3),
                                 "gops": 2.0 * macs / ((t_conv + t_pack) * 1e-3) / 1e9,
                                 "frac": sums["roofline_s_burst"] / (t_conv * 1e-3), "frac_sustained": sums["roofline_s_sustained"] / (t_conv * 1e-3),
                                 "hbm_bound_layers": sums["hbm_bound_layers"],
                                 "pack_frac_hbm": (x.numel() * 4 + runner.bufs[net.in_name].numel() * 4) / (t_pack * 1e-3) / pk["hbm"]}
    del runner, x
    # ---- runs of same-shaped layers as one launch (bitserial_conv2d_tc_chain) against one launch per layer
    chain_rows = []
    for b in (16, 64):
        cnet, cseed = make_net("resnet18_body", b)
        cparams = wl.network_params(cnet, cseed)
        row = {"workload": f"resnet18_body_batch{b}_w2a2, conv layers only (warm L2, one CUDA graph per pass)"}
        for key, mode in (("per_layer", False), ("chains", True)):
            r = BitserialNet(cnet, cparams, ACT_SCALE, batch=b, engine="tc", chains=mode)
            with torch.cuda.stream(stream):
                r.run_layers()
                stream.synchronize()
                row[key + "_ms"] = graph_time(r.run_layers, reps=1, rounds=8)
            row[key + "_launches"] = len(r.units)
            del r
        auto = BitserialNet(cnet, cparams, ACT_SCALE, batch=b, engine="tc", chains="auto")
        row["auto_keeps_launches"] = len(auto.units)
        del auto
        chain_rows.append(row)
    out["layer_chains"] = chain_rows
    # ---- the whole mixed-precision classifier: floating-point stem and head around the headline stack
    from paper_2207_08820_b200.net import BitserialFullNet
    fnet = wl.resnet18_full(batch=args.batch)
    fparams = wl.full_network_params(fnet, 3000)
    images = torch.from_numpy(wl.full_network_input(fnet, 3000)).cuda()
    full = BitserialFullNet(fnet, fparams, batch=fnet.batch, engine="tc")
    with torch.cuda.stream(stream):
        full.forward(images)
        stream.synchronize()
        t_stem = graph_time(lambda: full.run_stem(images), reps=1, rounds=6)
        t_packf = graph_time(lambda: full.body.pack_input(full.stem_pool), reps=1, rounds=6)
        t_body = graph_time(full.body.run_layers, reps=1, rounds=8)
        t_head = graph_time(full.run_head, reps=1, rounds=6)
        t_all = graph_time(lambda: full.forward(images), reps=1, rounds=8)
    stem_flops = 2.0 * fnet.stem_macs_per_image() * fnet.batch
    fp32_peak = 2.0 * 128 * torch.cuda.get_device_properties(0).multi_processor_count * peaks["sm_max_mhz"] * 1e6
    out["resnet18_full"] = {"workload": f"resnet18_full_batch{fnet.batch}_224px: fp32 stem (7x7 s2 conv + 3x3 s2 max pool), quantise + pack, W2A2 body, fp32 head "
                                        "(average pool + 512 -> 1000 fully connected); warm L2, one CUDA graph per part",
                            "stem_ms": t_stem, "pack_ms": t_packf, "body_ms": t_body, "head_ms": t_head, "forward_ms": t_all,
                            "images_per_s": fnet.batch / (t_all * 1e-3), "stem_fp32_TFLOPs": stem_flops / (t_stem * 1e-3) / 1e12,
                            "stem_frac_fp32_fma_peak": stem_flops / (t_stem * 1e-3) / fp32_peak,
                            "fp32_fma_peak_TFLOPs": fp32_peak / 1e12, "body_only_images_per_s": fnet.batch / ((t_body + t_packf) * 1e-3)}
    launches += 0
    api.bs_check_status(stream)
    return out, launches


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
    chains = False if args.eager or args.chains == "off" else (True if args.chains == "on" else "auto")
    runner = BitserialNet(net, params, ACT_SCALE, batch=net.batch, engine=args.engine, chains=chains)

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
        # The timed loop: EXACTLY args.steps steps between two barriers.  It is repeated as whole rounds until at least
        # --min-timed-s of step time has been measured (every rank runs the same number of rounds: the count is fixed from
        # the first round's time, maximum over ranks); the reported times are means over all rounds, the spread is per step.
        all_events = []
        with ClockSampler(local) as clocks:
            rounds = 1
            r = 0
            while r < rounds:
                events = [[torch.cuda.Event(enable_timing=True) for _ in range(3)] for _ in range(args.steps)]
                barrier()
                for k in range(args.steps):
                    flush_l2()             # L2 flush between timed iterations (outside the event pairs)
                    step(events[k])
                barrier()
                all_events.extend(events)
                if r == 0 and args.min_timed_s > 0:
                    first = sum(e[0].elapsed_time(e[2]) for e in events) * 1e-3
                    first = replicas.max_over_ranks([first], torch.device("cuda", local))[0]
                    rounds = max(1, min(400, int(np.ceil(args.min_timed_s / max(first, 1e-6)))))
                r += 1
        events = all_events
        nsteps = len(events)
        step_ms = np.array([e[0].elapsed_time(e[2]) for e in events])
        t_pack = sum(e[0].elapsed_time(e[1]) for e in events) / nsteps
        t_conv = sum(e[1].elapsed_time(e[2]) for e in events) / nsteps
        t_step = float(step_ms.mean())
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

    configs, config_launches = None, 0
    if world == 1 and rank == 0 and not args.no_configs and not args.eager and args.workload == "resnet18_body" and not args.hw:
        configs, config_launches = measure_other_configs(torch, api, stream, args)

    t_step, t_e2e, t_conv, t_pack = replicas.max_over_ranks([t_step, t_e2e, t_conv, t_pack], torch.device("cuda", local))

    if rank == 0:
        macs = net.macs_per_image() * net.batch
        wops = wordops_per_image(net) * net.batch
        gops = 2.0 * macs * world / (t_step * 1e-3) / 1e9
        peaks, peak_kind = measured_peaks()
        sms = torch.cuda.get_device_properties(local).multi_processor_count
        popc_peak = POPC_PER_CLK_PER_SM * sms * peaks["sm_max_mhz"] * 1e6          # counts/s at the maximum SM clock
        popc_measured = api.bs_popc_rate(4096)
        # dense int8 = 2 x bf16 (nominal ratio); the conv kernels are timed 17 us at a time inside a millisecond step at the
        # maximum clock, so the burst figure is the denominator of `frac`; the sustained one is printed beside it
        int8_burst = 2.0 * peaks["bf16_tflops"]
        int8_sustained = 2.0 * peaks.get("bf16_tflops_sustained", peaks["bf16_tflops"])

        def popc_roofline(t_ms):
            a = wops / (t_ms * 1e-3)
            _, sums = layer_roofline(net, "popc", peaks, popc_peak / POPC_PER_WORDOP)
            return {"bound": "alu", "kernel": "bitserial_conv_kernel", "achieved": a * POPC_PER_WORDOP / 1e12, "peak": popc_peak / 1e12,
                    "unit": "Tpopc/s", "frac": a * POPC_PER_WORDOP / popc_peak, "traffic": None,
                    "peak_source": f"{POPC_PER_CLK_PER_SM} popc/clk/SM x {sms} SMs x {peaks['sm_max_mhz']:.0f} MHz ({peak_kind} clock); achieved = population "
                                   "counts EXECUTED per second: the 3:2 carry-save adder executes 2 counts per 3 popc32(AND) word operations of the plane-pair sum",
                    "frac_algorithmic": a / popc_peak, "achieved_algorithmic_Twordop_s": a / 1e12,
                    "frac_per_layer_roofline": sums["roofline_s_burst"] / (t_ms * 1e-3), "hbm_bound_layers": sums["hbm_bound_layers"],
                    "popc_pipe_measured": popc_measured / 1e12, "launches_per_step": len(net.layers),
                    "avg_launch_ms": t_ms / len(net.layers)}

        tc_traffic, tc_traffic_src = captured_traffic(net.name, net.batch)

        def tensor_roofline(t_ms):
            a = 2.0 * macs / (t_ms * 1e-3) / 1e12
            rows, sums = layer_roofline(net, "tc", peaks, popc_peak)
            return {"bound": "tensor", "kernel": "bitserial_conv_tc_persistent_kernel", "achieved": a, "peak": int8_burst,
                    "unit": "TOP/s", "frac": a / int8_burst, "peak_burst": int8_burst, "peak_sustained": int8_sustained,
                    "frac_sustained": a / int8_sustained,
                    # per layer max(t_tensor, t_hbm), summed over the stack, over the measured conv time
                    "frac_per_layer_roofline": sums["roofline_s_burst"] / (t_ms * 1e-3),
                    "frac_per_layer_roofline_sustained": sums["roofline_s_sustained"] / (t_ms * 1e-3),
                    "hbm_bound_layers": sums["hbm_bound_layers"], "algorithmic_bytes_per_launch": sums["bytes"] / len(net.layers),
                    "traffic": tc_traffic / len(net.layers) if tc_traffic else None, "traffic_source": tc_traffic_src,
                    "peak_source": f"2 x {peak_kind} bf16 cuBLAS TFLOP/s (nominal int8:bf16 ratio); burst figure (kernels of ~17 us inside a short step at the maximum clock)",
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
            "ms_per_step_stats": {"mean": t_step, "std": float(step_ms.std()), "min": float(step_ms.min()), "max": float(step_ms.max()),
                                  "rounds_of_K_steps": rounds, "steps_timed": nsteps, "timed_s": float(step_ms.sum()) * 1e-3},
            "roofline": roof,
            "pack": {"bound": "hbm", "ms": t_pack, "achieved": pack_bytes / (t_pack * 1e-3) / 1e9, "peak": peaks["hbm_gbs"],
                     "unit": "GB/s", "frac": pack_bytes / (t_pack * 1e-3) / 1e9 / peaks["hbm_gbs"],
                     "note": "54.6 MB input: a 12 us kernel, ramp and tail dominate; pack_large has the inputs larger than L2"},
            "e2e": {"value": 2.0 * macs * world / (t_e2e * 1e-3) / 1e9, "unit": UNIT, "ms_per_step": t_e2e, "overlap": "h2d of step k+1 beside the kernels of step k (two input buffers); L2 flush inside",
                    "h2d_bytes_per_step": in_bytes, "d2h_bytes_per_step": out_host.numel() * 4},
            "gpu_launches": runner.launches_per_forward * nsteps,
            "clocks": clocks.summary(),
        }
        line["config"]["engine"] = args.engine
        line["config"]["conv_launches_per_step"] = len(runner.units)
        if t_conv_other is not None:
            alt = popc_roofline(t_conv_other) if other == "popc" else tensor_roofline(t_conv_other)
            alt["engine"] = other
            alt["conv_ms"] = t_conv_other
            line["other_engine"] = alt
        popc_frac = (roof if args.engine == "popc" else line.get("other_engine", {})).get("frac")
        tc_frac = (roof if args.engine == "tc" else line.get("other_engine", {})).get("frac")
        line["target_0p60_of_roofline"] = {
            "popcount_kernel_frac_executed": popc_frac, "tensor_core_kernel_frac": tc_frac,
            "statement": "the bit-serial (popcount) conv kernel is measured against the popc-pipe peak on executed counts; the tensor-core "
                         "formulation, adopted because it is faster in absolute time, is measured against the int8 tensor peak and does not reach 0.60 of it"}
        if configs is not None:
            line["configs"] = configs
            line["gpu_launches"] += config_launches
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
    ap.add_argument("--min-timed-s", type=float, default=0.5, help="the K-step timed loop is repeated (rounds) until this much time has been "
                    "measured, so that clock samples see the GPU under load; 0 = a single round")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="resnet18_body", choices=["resnet18_body", "detection_backbone", "resnet50_body", "vgg16_ssd_body", "bitwidth_sweep", "gemm_sweep"])
    ap.add_argument("--hw", type=int, default=0, help="side of the first packed tensor (default: the workload's own; the paper's 320 / 352 px "
                    "detection inputs are --workload detection_backbone --hw 160 / 176)")
    ap.add_argument("--batch", type=int, default=0, help="images per GPU (default: 64 / 16 / 32 / 8 as the workload defines)")
    ap.add_argument("--ref-images", type=int, default=2, help="images per step of the reference arm (bounded CPU sample)")
    ap.add_argument("--cpu-baseline-images", type=int, default=64, help="images of the one oracle pass timed beside the GPU run")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-configs", action="store_true", help="leave out the compact measurements of the other workloads")
    ap.add_argument("--engine", default="tc", choices=["popc", "tc"],
                    help="popc: popcount kernels on the integer pipes; tc: exact int8 tensor-core formulation")
    ap.add_argument("--chains", default="auto", choices=["auto", "on", "off"], help="runs of same-shaped layers as one launch: timed at set-up and "
                    "kept where faster (auto), always, or never; --eager implies off")
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
