"""GPU parity on layer stacks: every activation tensor of the residual stack and of the detection-shaped
stack, free-running on both sides from the same seeded fp32 input (no tensor crosses from the GPU to the
oracle).  Tolerance as for single layers; zero mismatches are expected."""
import numpy as np
import pytest
import torch

import oracle
from oracle import network as onet
from paper_2207_08820_b200 import api, workloads as wl
from paper_2207_08820_b200.net import BitserialNet
from gpu_util import Guarded, dev

pytestmark = pytest.mark.gpu

ACT_SCALE = 0.25


def compare_stack(net, batch, seed, sample=None, graph=False, engine="popc"):
    params = wl.network_params(net, seed)
    x = wl.network_input(net, seed, ACT_SCALE, batch=batch)
    runner = BitserialNet(net, params, ACT_SCALE, batch=batch, engine=engine)
    guard = Guarded()                      # every activation buffer of the runner gets guard words around it
    for name, buf in list(runner.bufs.items()):
        runner.bufs[name] = guard.empty(tuple(buf.shape), fill=0)
    xd = dev(x)
    if graph:
        runner.capture(xd)
        runner.replay(xd)
    else:
        runner.forward(xd)
    api.bs_check_status()
    guard.check()
    idx = list(range(batch)) if sample is None else sample
    want = onet.run_stack(net, params, x[idx], ACT_SCALE)
    levels = set()
    for name in net.tensor_shapes():
        got = runner.unpacked(name).cpu().numpy()[idx]
        diff = np.abs(got.astype(np.int32) - want[name].astype(np.int32))
        assert diff.max() <= 1, name
        assert (diff != 0).mean() <= 1e-4, name
        levels |= set(np.unique(want[name]).tolist())
    assert levels == {0, 1, 2, 3}
    out = want[net.out_name]
    assert len(np.unique(out)) >= 3          # the stack does not collapse to a constant


def test_resnet18_body_small_batch():
    compare_stack(wl.resnet18_body(2), 2, seed=3000)


def test_detection_backbone_small():
    compare_stack(wl.detection_backbone(1, hw=64), 1, seed=4000)


def test_resnet18_body_full_batch_graph_sampled():
    """Batch 64 through the CUDA-graph path the benchmark times; the oracle runs three sampled images."""
    compare_stack(wl.resnet18_body(64), 64, seed=3000, sample=[0, 31, 63], graph=True)


def test_detection_backbone_full_size_sampled():
    compare_stack(wl.detection_backbone(16), 16, seed=4000, sample=[0, 15], graph=True)


def test_resnet18_body_tensor_core_small_batch():
    compare_stack(wl.resnet18_body(2), 2, seed=3000, engine="tc")


def test_detection_backbone_tensor_core_small():
    compare_stack(wl.detection_backbone(1, hw=64), 1, seed=4000, engine="tc")


def test_resnet18_body_tensor_core_full_batch_graph_sampled():
    compare_stack(wl.resnet18_body(64), 64, seed=3000, sample=[0, 31, 63], graph=True, engine="tc")


def test_detection_backbone_tensor_core_full_size_sampled():
    compare_stack(wl.detection_backbone(16), 16, seed=4000, sample=[0, 15], graph=True, engine="tc")


@pytest.mark.parametrize("engine", ["popc", "tc"])
def test_resnet50_body_small(engine):
    """Bottleneck stack (1x1 / 3x3 / 1x1 with 4x widening, projection shortcuts) at a reduced resolution."""
    compare_stack(wl.resnet50_body(2, hw=16), 2, seed=6000, engine=engine)


@pytest.mark.parametrize("engine", ["popc", "tc"])
def test_vgg16_ssd_body_small(engine):
    """Plain 3x3 stack with odd intermediate widths (40 -> 20 -> 10 -> 5 -> 3) at a reduced resolution."""
    compare_stack(wl.vgg16_ssd_body(1, hw=40), 1, seed=7000, engine=engine)


def test_vgg16_ssd_body_full_resolution_sampled():
    """300 px: widths 300/150/75/38/19 (odd and even) through the tensor-core engine, one image checked."""
    compare_stack(wl.vgg16_ssd_body(2), 2, seed=7000, sample=[1], graph=True, engine="tc")


def test_resnet50_body_full_batch_sampled():
    """Batch 32 at 56 px (the configuration `bench.py --workload resnet50_body` times): wide 1x1 chunks, streamed deep
    reductions and projection shortcuts on the second stream, two images checked against the oracle."""
    compare_stack(wl.resnet50_body(32), 32, seed=6000, sample=[0, 31], graph=True, engine="tc")


def test_detection_backbone_352px_input():
    """The paper's 352 px detection input: first packed tensor 176 px, widths 176 / 88 / 44 / 22 / 11."""
    compare_stack(wl.detection_backbone(1, hw=176), 1, seed=4000, engine="tc")
