"""Per-layer times of a layer stack on one GPU.

    python -m paper_2207_08820_b200.layer_times resnet18_body [batch] [engine]

Every layer is launched alone in three ways, each inside a CUDA graph and timed with CUDA events (warm L2, best of four replays):
once; eight times back to back; eight times back to back as launches chained by programmatic dependent launch (the way the stack
runs them; tensor-core engine only).  The last column is the layer's arithmetic over the chained time.  Host logic only.
"""
from __future__ import annotations

import sys

import torch

from . import api, workloads as wl
from .net import BitserialNet

STACKS = {"resnet18_body": (wl.resnet18_body, 64, 3000), "detection_backbone": (wl.detection_backbone, 16, 4000),
          "resnet50_body": (wl.resnet50_body, 32, 6000), "vgg16_ssd_body": (wl.vgg16_ssd_body, 8, 7000)}
REPS = 8


def main(argv) -> int:
    name = argv[1] if len(argv) > 1 else "resnet18_body"
    make, batch, seed = STACKS[name]
    if len(argv) > 2:
        batch = int(argv[2])
    engine = argv[3] if len(argv) > 3 else "tc"
    net = make(batch)
    params = wl.network_params(net, seed)
    x = torch.from_numpy(wl.network_input(net, seed, 0.25, batch=batch)).cuda()
    runner = BitserialNet(net, params, 0.25, batch=batch, engine=engine, chains=False)
    runner.forward(x)
    api.bs_check_status()
    stream = torch.cuda.Stream()
    shapes = net.tensor_shapes()
    total_single = total_chained = 0.0
    with torch.cuda.stream(stream):
        for item in runner.layers:
            L = item["spec"]
            _, P, Q = shapes[L.dst]
            macs = batch * P * Q * L.O * L.C * L.k * L.k
            times = []
            for reps, chained in ((1, False), (REPS, False), (REPS, True)):
                runner.run_layer(item, chained=False)
                stream.synchronize()
                graph = torch.cuda.CUDAGraph()
                with torch.cuda.graph(graph, stream=stream):
                    for _ in range(reps):
                        runner.run_layer(item, chained=chained)
                best = float("inf")
                for k in range(6):
                    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                    e0.record(stream)
                    graph.replay()
                    e1.record(stream)
                    e1.synchronize()
                    if k >= 2:
                        best = min(best, e0.elapsed_time(e1) * 1e3 / reps)
                times.append(best)
            t1, tr, tc = times
            total_single += t1
            total_chained += tc
            print(f"{L.name:14s} C{L.C:5d} O{L.O:5d} k{L.k} s{L.stride} {P:3d}x{Q:<3d} res={int(bool(L.res))}  single {t1:6.2f} us  x{REPS} {tr:6.2f}  "
                  f"chained {tc:6.2f} us  {2 * macs / tc / 1e6:7.1f} TOP/s")
    print(f"sum of single launches {total_single:.1f} us, sum of chained launches {total_chained:.1f} us")
    api.bs_check_status()
    return 0


if __name__ == "__main__":
    sys.exit(main(sys.argv))
