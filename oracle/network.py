"""Oracle-side execution of a layer stack (TEST INFRASTRUCTURE ONLY).

Runs every layer as: direct integer convolution on unpacked codes, then the
requantisation epilogue, in the order the stack lists them.  The stack
description is duck-typed (objects with ``layers``, ``in_name``, ``a_bits`` and
per-layer ``src/dst/res/...`` attributes); nothing from the GPU package is
imported here.
"""
from __future__ import annotations

from typing import Dict

import numpy as np

from . import UNSIGNED, avgpool_codes, conv2d_f32, conv2d_i32, fc_f32, maxpool2d_f32, quantize, requantize


def run_stack(net, params: Dict[str, Dict], x_fp32: np.ndarray, act_scale: float,
              keep_acc: bool = False) -> Dict[str, np.ndarray]:
    """Returns {tensor name: int8 codes NCHW} for every activation tensor of the stack
    (and ``acc:<layer>`` int32 accumulators when ``keep_acc``)."""
    shapes = net.tensor_shapes()
    n = x_fp32.shape[0]
    t: Dict[str, np.ndarray] = {net.in_name: quantize(x_fp32, act_scale, net.a_bits, UNSIGNED)}
    for L in net.layers:
        p = params[L.name]
        src = t[L.src][:, :L.C]
        acc = conv2d_i32(src, p["w"], stride=L.stride, pad=L.pad)
        res = t[L.res][:, :L.O] if L.res else None
        codes = requantize(acc, p["scale"], p["bias"], L.relu, net.a_bits, UNSIGNED,
                           res=res, res_scale=L.res_scale)
        if L.dst not in t:
            c_total, P, Q = shapes[L.dst]
            t[L.dst] = np.zeros((n, c_total, P, Q), dtype=np.int8)
        t[L.dst][:, L.dst_c_offset:L.dst_c_offset + L.O] = codes
        if keep_acc:
            t["acc:" + L.name] = acc
    return t


def run_full(net, params: Dict[str, Dict], images: np.ndarray) -> Dict[str, np.ndarray]:
    """Whole classifier (duck-typed ``FullNetSpec``): floating-point stem -> quantiser -> quantised body -> floating-point head.
    Returns every tensor: ``stem_conv``, ``stem_pool`` (float32), the body's code tensors, ``pooled`` and ``logits``."""
    t: Dict[str, np.ndarray] = {}
    t["stem_conv"] = conv2d_f32(images, params["stem"]["w"], params["stem"]["bias"], stride=2, pad=3, relu=True)
    t["stem_pool"] = maxpool2d_f32(t["stem_conv"], 3, 2, 1)
    t.update(run_stack(net.body, params, t["stem_pool"], net.stem_act_scale))
    last = t[net.body.out_name]
    inv = np.float32(np.float32(net.body_act_scale) / np.float32(last.shape[2] * last.shape[3]))
    t["pooled"] = avgpool_codes(last, float(inv))
    t["logits"] = fc_f32(t["pooled"], params["fc"]["w"], params["fc"]["bias"])
    return t
