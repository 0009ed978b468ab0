"""Per-CTA timeline of the tensor-core kernels (tuning builds only).

A library built with ``BS_EXTRA_NVCC_FLAGS=-DBS_TUNING python -m paper_2207_08820_b200.build --force`` records, for the first
148 CTAs of a launch and the first 24 pixel tiles of each, the SM cycle counter at the hand-offs between the kernel's roles
(packed tile requested / landed, expansion begin / end, MMA issue begin / end, epilogue begin / end; per channel chunk instead of
per tile for the kernel that streams its filters).  This tool runs chosen layers
of a layer stack once and prints those timelines:

    python -m paper_2207_08820_b200.timeline resnet18_body 0,7 [cta,cta,...]

Host logic only; the normal library has no such entry point and the tool says so.
"""
from __future__ import annotations

import ctypes
import sys

import numpy as np
import torch

from . import api, workloads as wl
from ._lib import lib
from .net import BitserialNet

EVENTS = ["START", "SETUP", "PDL", "WGT", "LOAD", "XBEG", "XEND", "MBEG", "MEND", "EBEG", "EEND", "END", "E_LD", "E_CMP", "E_ST", "E_LOOP",
          "M_ISSUED", "X_DONE0", "X_BEG0"]
STACKS = {"resnet18_body": (wl.resnet18_body, 64, 3000), "detection_backbone": (wl.detection_backbone, 16, 4000),
          "resnet50_body": (wl.resnet50_body, 32, 6000), "vgg16_ssd_body": (wl.vgg16_ssd_body, 8, 7000)}


def main(argv) -> int:
    name = argv[1] if len(argv) > 1 else "resnet18_body"
    layers = [int(v) for v in argv[2].split(",")] if len(argv) > 2 else [0]
    ctas = [int(v) for v in argv[3].split(",")] if len(argv) > 3 else [0, 147]
    L = lib()
    if not hasattr(L, "bs_tc_trace_read"):
        print("this library was not built with -DBS_TUNING: no timeline is recorded")
        return 1
    L.bs_tc_trace_read.restype = ctypes.c_int
    L.bs_tc_trace_read.argtypes = [ctypes.c_void_p, ctypes.c_int]
    make, batch, seed = STACKS[name]
    net = make(batch)
    params = wl.network_params(net, seed)
    x = torch.from_numpy(wl.network_input(net, seed, 0.25)).cuda()
    runner = BitserialNet(net, params, 0.25, batch=batch, engine="tc")
    runner.forward(x)
    api.bs_check_status()
    buf = np.zeros((148, 24, 24), dtype=np.int64)
    for li in layers:
        item = runner.layers[li]
        for _ in range(3):
            runner.run_layer(item, chained=False)
        L.bs_tc_trace_read(buf.ctypes.data, 1)
        runner.run_layer(item, chained=False)
        L.bs_tc_trace_read(buf.ctypes.data, 1)
        spec = item["spec"]
        print(f"layer {li} {spec.name}: C {spec.C} O {spec.O} k {spec.k} stride {spec.stride}")
        for c in ctas:
            t0 = buf[c, 0, 0]
            if t0 == 0:
                print(f"  CTA {c}: no timeline (fewer CTAs in this launch)")
                continue
            if buf[c, 3, 0] == 0:
                # the streaming kernel (one pixel-tile group per CTA, filters fetched chunk by chunk): one line per channel chunk
                rel = lambda e, t=0: buf[c, e, t] - t0
                print(f"  CTA {c} (filters streamed): ends at {rel(11)} cycles; tables built {rel(1)}, packed tile landed {rel(2)}, "
                      f"expansion finished {rel(13)}, accumulators ready {rel(9)}, epilogue done {rel(10)}")
                for t in range(24):
                    if buf[c, 5, t] == 0:
                        break
                    print(f"    chunk {t}: filters requested {rel(4, t)}  expand {rel(5, t)}..{rel(6, t)}  mma issue {rel(7, t)}..{rel(8, t)}")
                continue
            print(f"  CTA {c}: ends at {buf[c, 11, 0] - t0} cycles; set-up {buf[c, 1, 0] - t0}, filters landed {buf[c, 3, 0] - t0}")
            for t in range(24):
                if buf[c, 4, t] == 0 and buf[c, 5, t] == 0:
                    break
                rel = lambda e: buf[c, e, t] - t0
                print(f"    tile {t}: load {rel(4)}  expand {rel(5)}..{rel(6)} (first chunk {rel(18)}..{rel(17)})  "
                      f"mma {rel(7)}..{rel(8)} (first chunk issued {rel(16)})  epilogue {rel(9)}..{rel(10)} (accumulators read {rel(12)})")
        ends = (buf[:, 11, 0] - buf[:, 0, 0])[buf[:, 0, 0] != 0]
        if ends.size:
            print(f"  CTA durations: min {ends.min()} median {int(np.median(ends))} max {ends.max()} over {ends.size} CTAs")
    return 0


if __name__ == "__main__":
    sys.exit(main(sys.argv))
