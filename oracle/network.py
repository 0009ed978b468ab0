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

from . import UNSIGNED, conv2d_i32, quantize, requantize


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
