"""The N > 1 host path (batch sharding, barrier, max-over-ranks timing) on CPU with gloo, world size 2."""
import os
import socket

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2207_08820_b200 import replicas, workloads as wl


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        b, e = replicas.shard_range(7, rank, world)
        net = wl.resnet18_body(2)
        x = wl.network_input(net, replicas.rank_seed(3000, rank), 0.25, batch=1)
        dist.barrier()
        times = replicas.max_over_ranks([10.0 + rank, 5.0 - rank], torch.device("cpu"))
        dist.barrier()
        out.put((rank, b, e, float(x.sum()), times))
    finally:
        dist.destroy_process_group()


def test_two_replicas_shard_and_reduce():
    world = 2
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, world, port, q)) for r in range(world)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=120) for _ in range(world))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    (r0, b0, e0, s0, t0), (r1, b1, e1, s1, t1) = res
    assert (b0, e0, b1, e1) == (0, 4, 4, 7)                 # 7 images over 2 ranks: 4 + 3, contiguous, disjoint
    assert s0 != s1                                          # every replica draws its own batch
    assert t0 == t1 == [11.0, 5.0]                           # max over ranks, seen identically by all ranks


def test_shard_range_covers_everything():
    for total in (0, 1, 5, 64, 1000):
        for world in (1, 2, 3, 8):
            spans = [replicas.shard_range(total, r, world) for r in range(world)]
            assert spans[0][0] == 0 and spans[-1][1] == total
            assert all(spans[i][1] == spans[i + 1][0] for i in range(world - 1))
            sizes = [e - b for b, e in spans]
            assert max(sizes) - min(sizes) <= 1
    with pytest.raises(ValueError):
        replicas.shard_range(4, 2, 2)
    assert replicas.aggregate_throughput(64, 8, 4.0) == 64 * 8 / 4e-3
