"""Seeded synthetic inputs and layer tables for the bit-serial convolution workloads.

This module holds shapes, random draws and parameter recipes only: no
quantisation, packing, convolution or requantisation arithmetic lives here, so
the GPU library and any independent checker can both consume its outputs.

Everything is numpy; code tensors are int8 (NCHW activations, OIHW weights,
row-major matrices).  Sign conventions: 0 unsigned, 1 two's complement,
2 bipolar {-1,+1} (1 bit).
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Dict, List, Optional, Tuple

import numpy as np

UNSIGNED, SIGNED, BIPOLAR = 0, 1, 2


def code_range(bits: int, sign: int) -> Tuple[int, int]:
    if sign == SIGNED:
        return -(1 << (bits - 1)), (1 << (bits - 1)) - 1
    if sign == BIPOLAR:
        return -1, 1
    return 0, (1 << bits) - 1


def rand_codes(rng: np.random.Generator, shape, bits: int, sign: int) -> np.ndarray:
    """Codes uniform over the representable range (bipolar: +-1 with p = 0.5)."""
    if sign == BIPOLAR:
        return (2 * rng.integers(0, 2, size=shape, dtype=np.int8) - 1).astype(np.int8)
    lo, hi = code_range(bits, sign)
    return rng.integers(lo, hi + 1, size=shape, dtype=np.int8)


def rand_weights_zero_mean(rng: np.random.Generator, shape, bits: int, sign: int) -> np.ndarray:
    """Weights over the full code range with zero mean: the most negative code of a two's-complement
    range has no positive partner, so it and its neighbour get half the probability of the others,
    re-balanced so that the expectation is exactly zero (2 bits: p(-2), p(-1), p(0), p(1) = 1/7, 1/7,
    2/7, 3/7).  Keeps every filter's sum near zero, so accumulators do not inherit the common-mode
    brightness of a pixel and deep stacks keep all activation levels in use."""
    if sign != SIGNED or bits < 2:
        return rand_codes(rng, shape, bits, sign)
    lo, hi = code_range(bits, sign)
    vals = np.arange(lo, hi + 1)
    p = np.ones(len(vals))
    p[0] = p[1] = 0.5
    # tilt the non-negative side so that sum(p * v) = 0
    neg = float((p * vals)[vals < 0].sum())
    pos = float((p * vals)[vals > 0].sum())
    p[vals > 0] *= -neg / pos
    p /= p.sum()
    return rng.choice(vals, size=shape, p=p).astype(np.int8)


def weight_sign(w_bits: int) -> int:
    """Signed weights; 1-bit signed weights are bipolar."""
    return BIPOLAR if w_bits == 1 else SIGNED


def float_activations(rng: np.random.Generator, shape, bits: int, act_scale: float) -> np.ndarray:
    """fp32 activations whose unsigned b-bit codes at step ``act_scale`` are uniform over all levels."""
    hi = (1 << bits) - 1
    u = rng.uniform(-0.5, hi + 0.5, size=shape)
    return (u * act_scale).astype(np.float32)


def code_moments(bits: int, sign: int) -> Tuple[float, float]:
    """Mean and variance of a code drawn uniformly over its range."""
    if sign == BIPOLAR:
        return 0.0, 1.0
    lo, hi = code_range(bits, sign)
    v = np.arange(lo, hi + 1, dtype=np.float64)
    return float(v.mean()), float(v.var())


def calibrated_scale_bias(w_codes: np.ndarray, a_bits: int, a_sign: int, out_bits: int,
                          res_scale: float = 0.0, res_bits: int = 0) -> Tuple[np.ndarray, np.ndarray]:
    """Per-filter scale and bias that spread requantised codes over all levels.

    For activations with mean m and variance v per element, an accumulator of
    filter o has mean m * sum(w_o) and variance v * sum(w_o^2).  The recipe maps
    that distribution to unit spread around the middle output level (and
    re-centres for an optional residual term of mean level), standing in for the
    calibration pass that produces a scale and bias per layer.
    """
    m, v = code_moments(a_bits, a_sign)
    w = w_codes.reshape(w_codes.shape[0], -1).astype(np.float64)
    mu = m * w.sum(axis=1)
    sigma = np.sqrt(np.maximum(v * (w * w).sum(axis=1), 1.0))
    mid = ((1 << out_bits) - 1) / 2.0
    scale = 1.0 / sigma
    bias = mid - mu * scale
    if res_scale != 0.0:
        bias = bias - res_scale * (((1 << res_bits) - 1) / 2.0)
    return scale.astype(np.float32), bias.astype(np.float32)


# --------------------------------------------------------------------------------------
# Single-layer workloads
# --------------------------------------------------------------------------------------

def single_conv_case(seed: int = 0, N: int = 1, C: int = 64, H: int = 56, W: int = 56, O: int = 64,
                     k: int = 3, stride: int = 1, pad: int = 1, a_bits: int = 2, w_bits: int = 2,
                     a_sign: int = UNSIGNED, w_sign: Optional[int] = None, out_bits: int = 2,
                     calibrated: bool = False) -> Dict:
    """One conv layer.  Defaults: 3x3, stride 1, pad 1, 1x64x56x56 unsigned 2-bit
    activations, 64 signed 2-bit filters, scale ~ U(0.01, 0.1), bias ~ N(0, 1), ReLU,
    2-bit output, seed 0."""
    rng = np.random.default_rng(seed)
    if w_sign is None:
        w_sign = weight_sign(w_bits)
    x = rand_codes(rng, (N, C, H, W), a_bits, a_sign)
    w = rand_codes(rng, (O, C, k, k), w_bits, w_sign)
    if calibrated:
        scale, bias = calibrated_scale_bias(w, a_bits, a_sign, out_bits)
    else:
        scale = rng.uniform(0.01, 0.1, size=O).astype(np.float32)
        bias = rng.normal(0.0, 1.0, size=O).astype(np.float32)
    return dict(x=x, w=w, scale=scale, bias=bias, N=N, C=C, H=H, W=W, O=O, R=k, S=k, stride=stride,
                pad=pad, a_bits=a_bits, a_sign=a_sign, w_bits=w_bits, w_sign=w_sign, relu=True,
                out_bits=out_bits, out_sign=UNSIGNED)


GEMM_SWEEP_MN = (256, 1024, 4096)
GEMM_SWEEP_K = (576, 2304, 4608)


def gemm_case(M: int, N: int, K: int, seed: int, a_bits: int = 2, a_sign: int = UNSIGNED,
              w_bits: int = 1, w_sign: int = BIPOLAR) -> Dict:
    """Matrix product in im2col form: unsigned 2-bit rows times 1-bit bipolar filters by default."""
    rng = np.random.default_rng(seed)
    a = rand_codes(rng, (M, K), a_bits, a_sign)
    w = rand_codes(rng, (N, K), w_bits, w_sign)
    return dict(a=a, w=w, M=M, N=N, K=K, a_bits=a_bits, a_sign=a_sign, w_bits=w_bits, w_sign=w_sign)


def gemm_sweep_seed(M: int, K: int) -> int:
    return 2000 + GEMM_SWEEP_MN.index(M) * 3 + GEMM_SWEEP_K.index(K)


BITWIDTH_SWEEP = ((1, 1), (1, 2), (2, 2), (2, 3), (3, 3))   # (w_bits, a_bits)


def bitwidth_sweep_case(w_bits: int, a_bits: int, N: int = 32, C: int = 256, H: int = 28, O: int = 256) -> Dict:
    seed = 5000 + BITWIDTH_SWEEP.index((w_bits, a_bits)) if (w_bits, a_bits) in BITWIDTH_SWEEP else 5999
    return single_conv_case(seed=seed, N=N, C=C, H=H, W=H, O=O, k=3, stride=1, pad=1, a_bits=a_bits,
                            w_bits=w_bits, out_bits=a_bits, calibrated=True)


# --------------------------------------------------------------------------------------
# Layer stacks
# --------------------------------------------------------------------------------------

@dataclass
class ConvSpec:
    """One quantised conv layer of a stack.  ``src``/``dst``/``res`` name activation tensors;
    the layer writes channels [dst_c_offset, dst_c_offset + O) of ``dst`` (concatenation for free)."""
    name: str
    src: str
    dst: str
    C: int
    O: int
    k: int
    stride: int
    pad: int
    relu: bool = True
    res: Optional[str] = None
    res_scale: float = 0.0
    dst_c_offset: int = 0


@dataclass
class NetSpec:
    name: str
    batch: int
    in_name: str
    in_shape: Tuple[int, int, int]            # (C, H, W) of the first packed tensor
    layers: List[ConvSpec] = field(default_factory=list)
    a_bits: int = 2
    w_bits: int = 2
    out_name: str = ""

    def tensor_shapes(self) -> Dict[str, Tuple[int, int, int]]:
        """(C_total, H, W) of every activation tensor, concatenation targets included."""
        shapes = {self.in_name: self.in_shape}
        for L in self.layers:
            _, H, W = shapes[L.src]
            P = (H + 2 * L.pad - L.k) // L.stride + 1
            Q = (W + 2 * L.pad - L.k) // L.stride + 1
            c_hi = L.dst_c_offset + L.O
            if L.dst in shapes:
                c0, p0, q0 = shapes[L.dst]
                assert (p0, q0) == (P, Q), L.name
                shapes[L.dst] = (max(c0, c_hi), P, Q)
            else:
                shapes[L.dst] = (c_hi, P, Q)
        return shapes

    def macs_per_image(self) -> int:
        shapes = self.tensor_shapes()
        total = 0
        for L in self.layers:
            _, P, Q = shapes[L.dst]
            total += P * Q * L.O * L.C * L.k * L.k
        return total


RES_SCALE = 0.5   # step ratio applied to the residual codes in the epilogue


def resnet18_body(batch: int = 64, hw: int = 56) -> NetSpec:
    """conv2_x .. conv5_x of an 18-layer residual network at 224 px input: four stages of two
    basic blocks (3x3 convs; widths 64/128/256/512; stages 3-5 start with a stride-2 3x3 conv and
    a 1x1 stride-2 projection shortcut).  The stem and classifier stay in floating point and are
    not part of this stack."""
    net = NetSpec(name="resnet18_body", batch=batch, in_name="x0", in_shape=(64, hw, hw))
    cur, c_in = "x0", 64
    for si, c in enumerate((64, 128, 256, 512)):
        for b in range(2):
            stride = 2 if (si > 0 and b == 0) else 1
            tag = f"s{si + 2}b{b}"
            mid, out = f"{tag}_mid", f"{tag}_out"
            shortcut = cur
            if stride != 1 or c_in != c:
                shortcut = f"{tag}_sc"
                net.layers.append(ConvSpec(f"{tag}_down", cur, shortcut, c_in, c, 1, stride, 0, relu=False))
            net.layers.append(ConvSpec(f"{tag}_conv1", cur, mid, c_in, c, 3, stride, 1))
            net.layers.append(ConvSpec(f"{tag}_conv2", mid, out, c, c, 3, 1, 1, res=shortcut, res_scale=RES_SCALE))
            cur, c_in = out, c
    net.out_name = cur
    return net


def resnet50_body(batch: int = 32, hw: int = 56) -> NetSpec:
    """conv2_x .. conv5_x of a 50-layer residual network at 224 px input: stages of 3/4/6/3 bottleneck blocks
    (1x1 c_in -> c, 3x3 c -> c carrying the stride, 1x1 c -> 4c + shortcut; c = 64/128/256/512), a 1x1 projection
    shortcut in the first block of every stage.  The first packed tensor is the 64-channel output of the
    floating-point stem; stem and classifier are not part of the stack."""
    net = NetSpec(name="resnet50_body", batch=batch, in_name="x0", in_shape=(64, hw, hw))
    cur, c_in = "x0", 64
    for si, (c, nblocks) in enumerate(((64, 3), (128, 4), (256, 6), (512, 3))):
        for b in range(nblocks):
            stride = 2 if (si > 0 and b == 0) else 1
            tag = f"s{si + 2}b{b}"
            shortcut = cur
            if b == 0:
                shortcut = f"{tag}_sc"
                net.layers.append(ConvSpec(f"{tag}_down", cur, shortcut, c_in, 4 * c, 1, stride, 0, relu=False))
            net.layers.append(ConvSpec(f"{tag}_1x1a", cur, f"{tag}_a", c_in, c, 1, 1, 0))
            net.layers.append(ConvSpec(f"{tag}_3x3", f"{tag}_a", f"{tag}_b", c, c, 3, stride, 1))
            net.layers.append(ConvSpec(f"{tag}_1x1b", f"{tag}_b", f"{tag}_out", c, 4 * c, 1, 1, 0, res=shortcut, res_scale=RES_SCALE))
            cur, c_in = f"{tag}_out", 4 * c
    net.out_name = cur
    return net


def vgg16_ssd_body(batch: int = 8, hw: int = 300) -> NetSpec:
    """The 3x3 conv layers of a 16-layer plain network at 300 px (single-shot-detector sized input) after its first,
    floating-point layer: conv1_2 (64 -> 64 at 300 px), then 2 x 128 at 150 px, 3 x 256 at 75 px, 3 x 512 at 38 px and
    3 x 512 at 19 px.  The 2x2 poolings between the groups are written as the stride of the next group's first
    conv (a pooling kernel is not part of the hot path; the layer shapes and MAC counts of the groups are kept)."""
    net = NetSpec(name="vgg16_ssd_body", batch=batch, in_name="x0", in_shape=(64, hw, hw))
    cur, c_in = "x0", 64
    groups = ((64, 1), (128, 2), (256, 3), (512, 3), (512, 3))
    for gi, (c, n) in enumerate(groups):
        for k in range(n):
            stride = 2 if (gi > 0 and k == 0) else 1
            name = f"g{gi + 1}_{k + 1}"
            net.layers.append(ConvSpec(name, cur, name + "_out", c_in, c, 3, stride, 1))
            cur, c_in = name + "_out", c
    net.out_name = cur
    return net


def detection_backbone(batch: int = 16, hw: int = 320) -> NetSpec:
    """Detection-backbone-shaped stack at 640 px input (first packed tensor 32 x 320 x 320): four
    stages, each a 3x3 stride-2 conv c/2 -> c followed by a cross-stage block with n bottlenecks:
    two 1x1 branches c -> c/2, n x [1x1 c/2 -> c/2, 3x3 c/2 -> c/2, + residual], concatenation,
    1x1 c -> c.  (c, n) = (64, 1), (128, 2), (256, 3), (512, 1)."""
    net = NetSpec(name="detection_backbone", batch=batch, in_name="x0", in_shape=(32, hw, hw))
    cur, c_in = "x0", 32
    for si, (c, n) in enumerate(((64, 1), (128, 2), (256, 3), (512, 1))):
        t = f"st{si}"
        h = c // 2
        net.layers.append(ConvSpec(f"{t}_down", cur, f"{t}_d", c_in, c, 3, 2, 1))
        cat = f"{t}_cat"
        net.layers.append(ConvSpec(f"{t}_cv2", f"{t}_d", cat, c, h, 1, 1, 0, dst_c_offset=h))
        net.layers.append(ConvSpec(f"{t}_cv1", f"{t}_d", f"{t}_y0", c, h, 1, 1, 0))
        y = f"{t}_y0"
        for b in range(n):
            last = b == n - 1
            net.layers.append(ConvSpec(f"{t}_b{b}_1x1", y, f"{t}_b{b}_m", h, h, 1, 1, 0))
            dst = cat if last else f"{t}_y{b + 1}"
            net.layers.append(ConvSpec(f"{t}_b{b}_3x3", f"{t}_b{b}_m", dst, h, h, 3, 1, 1, res=y, res_scale=RES_SCALE))
            y = dst
        net.layers.append(ConvSpec(f"{t}_cv3", cat, f"{t}_out", c, c, 1, 1, 0))
        cur, c_in = f"{t}_out", c
    net.out_name = cur
    return net


def network_params(net: NetSpec, seed: int) -> Dict[str, Dict]:
    """Random signed weights and calibrated scale/bias for every layer of a stack."""
    rng = np.random.default_rng(seed)
    ws = weight_sign(net.w_bits)
    params = {}
    for L in net.layers:
        w = rand_weights_zero_mean(rng, (L.O, L.C, L.k, L.k), net.w_bits, ws)
        scale, bias = calibrated_scale_bias(w, net.a_bits, UNSIGNED, net.a_bits,
                                            res_scale=L.res_scale if L.res else 0.0, res_bits=net.a_bits)
        params[L.name] = dict(w=w, scale=scale, bias=bias, w_sign=ws)
    return params


def network_input(net: NetSpec, seed: int, act_scale: float = 0.25, batch: Optional[int] = None) -> np.ndarray:
    """fp32 NCHW input whose codes at step ``act_scale`` are uniform over the unsigned range."""
    rng = np.random.default_rng(seed + 1)
    C, H, W = net.in_shape
    return float_activations(rng, (batch or net.batch, C, H, W), net.a_bits, act_scale)


# --------------------------------------------------------------------------------------
# Whole classifier: floating-point stem and head around the quantised body (mixed precision)
# --------------------------------------------------------------------------------------

@dataclass
class FullNetSpec:
    """An 18-layer residual classifier at ``hw`` x ``hw`` input: a floating-point stem (7x7 stride-2 convolution 3 -> 64 with
    bias and ReLU, 3x3 stride-2 max pool), the quantised body, and a floating-point head (global average pool of the last
    codes, fully connected layer to ``classes`` outputs).  ``stem_act_scale`` is the step of the quantiser between stem and
    body, ``body_act_scale`` the step of the body's codes (used by the average pool)."""
    name: str
    batch: int
    hw: int
    body: NetSpec
    classes: int = 1000
    stem_act_scale: float = 0.6
    body_act_scale: float = 0.25

    def stem_macs_per_image(self) -> int:
        return (self.hw // 2) ** 2 * 64 * 3 * 49

    def head_macs_per_image(self) -> int:
        return 512 * self.classes


def resnet18_full(batch: int = 64, hw: int = 224) -> FullNetSpec:
    return FullNetSpec(name="resnet18_full", batch=batch, hw=hw, body=resnet18_body(batch, hw // 4))


def full_network_params(net: FullNetSpec, seed: int) -> Dict[str, Dict]:
    """Body parameters as ``network_params``; stem and head weights drawn so that their outputs have unit scale."""
    params = network_params(net.body, seed)
    rng = np.random.default_rng(seed + 7)
    params["stem"] = dict(w=(rng.normal(0.0, 1.0, (64, 3, 7, 7)) / np.sqrt(147.0)).astype(np.float32),
                          bias=rng.normal(0.0, 0.1, 64).astype(np.float32))
    params["fc"] = dict(w=(rng.normal(0.0, 1.0, (net.classes, 512)) / np.sqrt(512.0)).astype(np.float32),
                        bias=rng.normal(0.0, 0.1, net.classes).astype(np.float32))
    return params


def full_network_input(net: FullNetSpec, seed: int, batch: Optional[int] = None) -> np.ndarray:
    """Normalised images: fp32 [batch, 3, hw, hw], standard normal (what mean/std normalisation of 8-bit images gives)."""
    rng = np.random.default_rng(seed + 2)
    return rng.normal(0.0, 1.0, (batch or net.batch, 3, net.hw, net.hw)).astype(np.float32)
