"""Seeded synthetic workloads: network shapes, random-init weights, inputs, arrival traces.

This module is *data only*.  It draws random numbers and lays out layer lists; it
performs none of the method's arithmetic (no convolution, no pooling, no softmax,
no compaction).  Both the CUDA library's tests and the CPU oracle consume the
arrays produced here, so the two sides see identical inputs without sharing code.

Layout conventions (the same on both sides):
  activations  NHWC  ``[B][H][W][C]``
  conv weights ``[Cout][kh][kw][Cin/groups]``  (K-major for the GEMM view
               M = B*Ho*Wo, N = Cout, K = kh*kw*Cin of a convolution mapped to a
               matrix product; paper Section II-C)
  FC weights   ``[n_classes][C]``

All arrays are float32.  For a ``bf16`` model every weight and input value is
already rounded to a bf16-representable number, so a consumer may narrow it
without further loss.

The paper evaluates on ImageNet with pretrained 4-exit ResNet-50 / Inception-v3
(Section IV, Benchmarks).  Neither is available offline; these generators stand in
with tensors of the same shapes (224x224x3 images, 1000 classes, three early exits
plus the final classifier) and random-init weights.
"""
from __future__ import annotations

import json
import os
from dataclasses import dataclass, field
from typing import List, Optional

import numpy as np

OP_CONV, OP_DWCONV, OP_MAXPOOL = 0, 1, 2
ACT_NONE, ACT_RELU, ACT_RELU6 = 0, 1, 2
FROM_PREV, FROM_STAGE_INPUT = -1, -2
NO_RESIDUAL = -1

_CAL_PATH = os.path.join(os.path.dirname(os.path.abspath(__file__)), "exit_calibration.json")


def _rng(seed: int, *stream: int) -> np.random.Generator:
    """Counter-based generator; ``stream`` separates independent draws under one seed."""
    return np.random.Generator(np.random.Philox(key=np.array([int(seed), _mix(stream)], dtype=np.uint64)))


def _mix(stream) -> int:
    h = 0x9E3779B97F4A7C15
    for s in stream:
        h = (h ^ (int(s) + 0x632BE59BD9B4E019 + (h << 6) + (h >> 2))) & 0xFFFFFFFFFFFFFFFF
    return h


def to_bf16_grid(a: np.ndarray) -> np.ndarray:
    """Round float32 values to the nearest bf16-representable float32 (library conversion)."""
    import torch

    return torch.from_numpy(np.ascontiguousarray(a, dtype=np.float32)).to(torch.bfloat16).to(torch.float32).numpy()


@dataclass
class Layer:
    op: int
    cin: int
    cout: int
    kh: int = 1
    kw: int = 1
    stride: int = 1
    pad: int = 0
    act: int = ACT_NONE
    input_from: int = FROM_PREV       # -1 previous layer (stage input for layer 0), -2 stage input, k>=0 layer k
    residual_from: int = NO_RESIDUAL  # -1 none, -2 stage input, k>=0 layer k; added before the activation
    weight: Optional[np.ndarray] = None   # [cout][kh][kw][cin/groups]; None for maxpool
    scale: Optional[np.ndarray] = None    # [cout] folded-BN scale
    bias: Optional[np.ndarray] = None     # [cout] folded-BN bias
    pad_w: int = -1                       # padding of the columns; -1 = the same as ``pad`` (which pads the rows)

    @property
    def groups(self) -> int:
        return self.cin if self.op == OP_DWCONV else 1


@dataclass
class Stage:
    layers: List[Layer]
    n_classes: int
    fc_weight: np.ndarray      # [n_classes][C]
    fc_bias: np.ndarray        # [n_classes]
    threshold: float
    always_exit: bool
    out_layer: int = -1        # index of the layer whose output leaves the stage (-1 = last)


@dataclass
class Model:
    name: str
    dtype: str                 # "f32" | "bf16"
    in_h: int
    in_w: int
    in_c: int
    stages: List[Stage]
    max_batch: int
    meta: dict = field(default_factory=dict)


def out_hw(h: int, w: int, l: Layer):
    pw = l.pad if l.pad_w < 0 else l.pad_w
    return (h + 2 * l.pad - l.kh) // l.stride + 1, (w + 2 * pw - l.kw) // l.stride + 1


def stage_shapes(model: Model):
    """Per stage: list of (H, W, C) for every layer output, plus the stage's in/out shape."""
    res = []
    h, w, c = model.in_h, model.in_w, model.in_c
    for st in model.stages:
        shapes = []
        for i, l in enumerate(st.layers):
            src = l.input_from
            if src == FROM_STAGE_INPUT or (src == FROM_PREV and i == 0):
                ih, iw, ic = h, w, c
            elif src == FROM_PREV:
                ih, iw, ic = shapes[i - 1]
            else:
                ih, iw, ic = shapes[src]
            assert ic == l.cin, (model.name, i, ic, l.cin)
            oh, ow = out_hw(ih, iw, l)
            shapes.append((oh, ow, l.cout))
        o = shapes[st.out_layer]
        res.append({"in": (h, w, c), "layers": shapes, "out": o})
        h, w, c = o
    return res


# ----------------------------------------------------------------------------- weights

def _conv(rng, op, cin, cout, k, stride, pad, act, *, gamma=1.0, jitter=True, bf16=False,
          input_from=FROM_PREV, residual_from=NO_RESIDUAL) -> Layer:
    cpg = 1 if op == OP_DWCONV else cin
    fan_in = k * k * cpg
    w = rng.standard_normal((cout, k, k, cpg), dtype=np.float32) * np.float32(np.sqrt(2.0 / fan_in))
    if jitter:
        scale = (gamma * rng.uniform(0.8, 1.2, size=cout)).astype(np.float32)
        bias = (0.05 * rng.standard_normal(cout)).astype(np.float32)
    else:
        scale = np.full(cout, gamma, dtype=np.float32)
        bias = np.zeros(cout, dtype=np.float32)
    if bf16:
        w = to_bf16_grid(w)
    return Layer(op, cin, cout, k, k, stride, pad, act, input_from, residual_from, w, scale, bias)


def _conv_hw(rng, cin, cout, kh, kw, stride, pad_h, pad_w, act, *, gamma=1.0, bf16=False, input_from=FROM_PREV,
             residual_from=NO_RESIDUAL) -> Layer:
    """A dense convolution with a kh x kw filter and per-axis padding (the factorised 1 x n / n x 1 filters of
    Inception-style towers)."""
    w = rng.standard_normal((cout, kh, kw, cin), dtype=np.float32) * np.float32(np.sqrt(2.0 / (kh * kw * cin)))
    scale = (gamma * rng.uniform(0.8, 1.2, size=cout)).astype(np.float32)
    bias = (0.05 * rng.standard_normal(cout)).astype(np.float32)
    if bf16:
        w = to_bf16_grid(w)
    return Layer(OP_CONV, cin, cout, kh, kw, stride, pad_h, act, input_from, residual_from, w, scale, bias, pad_w)


def head_weights(seed: int, stream: int, c: int, n_classes: int, alpha: float, bf16: bool):
    """FC head of one exit from its own random stream, so that it can be regenerated for another
    scale factor ``alpha`` without touching the backbone weights."""
    return _head(_rng(seed, 5000 + stream), c, n_classes, alpha, bf16)


def _head(rng, c, n_classes, alpha, bf16):
    w = rng.standard_normal((n_classes, c), dtype=np.float32) * np.float32(alpha / np.sqrt(c))
    b = (0.01 * rng.standard_normal(n_classes)).astype(np.float32)
    if bf16:
        w = to_bf16_grid(w)
    return w, b


def load_calibration() -> dict:
    """FC scale factors per model, written by ``oracle/calibrate_exit_scales.py`` (oracle only)."""
    if os.path.exists(_CAL_PATH):
        with open(_CAL_PATH) as f:
            return json.load(f)
    return {}


# ----------------------------------------------------------------------------- config 1

def tiny_ee_cnn(seed: int = 0, max_batch: int = 8, alphas=(3.0, 1.25, 2.0)) -> Model:
    """Three stages of two 3x3 convs (stride 1 then 2, pad 1), widths 16/32/64, fp32.

    Folded-BN scale 1 and bias 0, ReLU after every conv, exit head (GAP, FC to 10
    classes) after every stage, threshold 0.6 on exits 1-2, final exit always taken.
    """
    stages = []
    cin = 3
    for s, c in enumerate((16, 32, 64)):
        rng = _rng(seed, 100 + s)
        l0 = _conv(rng, OP_CONV, cin, c, 3, 1, 1, ACT_RELU, jitter=False)
        l1 = _conv(rng, OP_CONV, c, c, 3, 2, 1, ACT_RELU, jitter=False)
        fw, fb = _head(rng, c, 10, alphas[s], False)
        stages.append(Stage([l0, l1], 10, fw, np.zeros_like(fb), 0.6, s == 2))
        cin = c
    return Model("tiny_ee_cnn", "f32", 32, 32, 3, stages, max_batch, {"seed": seed})


# ----------------------------------------------------------------------------- config 2

def _bottleneck(rng, layers, cin, width, stride, project, bf16, in_idx):
    """Append one ResNet v1.5 bottleneck; ``in_idx`` is the layer index (or -2) of its input."""
    cout = 4 * width
    base = len(layers)
    layers.append(_conv(rng, OP_CONV, cin, width, 1, 1, 0, ACT_RELU, bf16=bf16, input_from=in_idx))
    layers.append(_conv(rng, OP_CONV, width, width, 3, stride, 1, ACT_RELU, bf16=bf16))
    if project:
        layers.append(_conv(rng, OP_CONV, cin, cout, 1, stride, 0, ACT_NONE, gamma=0.7, bf16=bf16, input_from=in_idx))
        res = base + 2
    else:
        res = in_idx
    layers.append(_conv(rng, OP_CONV, width, cout, 1, 1, 0, ACT_RELU, gamma=0.3, bf16=bf16,
                        input_from=base + 1, residual_from=res))
    return len(layers) - 1


def resnet50_ee(seed: int = 1, max_batch: int = 64, alphas=None, thresholds=(0.5, 0.6, 0.7),
                in_hw: int = 224, n_classes: int = 1000, blocks=(3, 4, 6, 3), width0: int = 64,
                dtype: str = "bf16") -> Model:
    """ResNet-50-shaped 4-exit backbone: stem 7x7 s2 + maxpool in stage 1, bottleneck stages
    [3,4,6,3] at widths 256/512/1024/2048, stride on the 3x3, 1x1 projection on the first block
    of each stage; exit heads (GAP + FC) after stages 1-3 plus the final head.

    ``in_hw``, ``blocks``, ``width0`` and ``n_classes`` shrink the network for fast tests;
    the defaults are the benchmark configuration.
    """
    bf16 = dtype == "bf16"
    if alphas is None:
        key = "resnet50_ee" if (in_hw, tuple(blocks), width0, n_classes, seed) == (224, (3, 4, 6, 3), 64, 1000, 1) else None
        alphas = load_calibration().get(key, {}).get("alphas", [6.0, 6.0, 6.0, 6.0]) if key else [6.0] * 4
    stages = []
    cin = 3
    for s, nb in enumerate(blocks):
        rng = _rng(seed, 200 + s)
        layers: List[Layer] = []
        width = width0 << s
        if s == 0:
            layers.append(_conv(rng, OP_CONV, 3, width0, 7, 2, 3, ACT_RELU, bf16=bf16))
            layers.append(Layer(OP_MAXPOOL, width0, width0, 3, 3, 2, 1))
            cin, idx = width0, 1
        else:
            idx = FROM_STAGE_INPUT
        for b in range(nb):
            idx = _bottleneck(rng, layers, cin, width, 2 if (b == 0 and s > 0) else 1, b == 0, bf16, idx)
            cin = 4 * width
        last = s == len(blocks) - 1
        fw, fb = head_weights(seed, 200 + s, cin, n_classes, alphas[s], bf16)
        stages.append(Stage(layers, n_classes, fw, fb, 1.0 if last else thresholds[s], last))
    return Model("resnet50_ee", dtype, in_hw, in_hw, 3, stages, max_batch,
                 {"seed": seed, "alphas": list(alphas), "thresholds": list(thresholds)})


# ----------------------------------------------------------------------------- config 3

def mobilenetv2_ee(seed: int = 2, max_batch: int = 32, alphas=None, threshold: float = 0.6,
                   in_hw: int = 224, n_classes: int = 1000, dtype: str = "bf16") -> Model:
    """MobileNetV2-shaped backbone with exits after inverted-residual blocks 4, 7 and 11.

    Stem 3x3 s2 -> 32; blocks (t, c, n, s) = (1,16,1,1) (6,24,2,2) (6,32,3,2) (6,64,4,2)
    (6,96,3,1) (6,160,3,2) (6,320,1,1); final 1x1 -> 1280 before the last head.  Expansion
    and depthwise convs use ReLU6, projection convs are linear, residual when stride 1 and
    Cin == Cout.  Stage split: [stem, b1-4] [b5-7] [b8-11] [b12-17, 1x1].
    """
    bf16 = dtype == "bf16"
    cfg = [(1, 16, 1, 1), (6, 24, 2, 2), (6, 32, 3, 2), (6, 64, 4, 2), (6, 96, 3, 1), (6, 160, 3, 2), (6, 320, 1, 1)]
    blocks = []
    cin = 32
    for t, c, n, s in cfg:
        for i in range(n):
            blocks.append((t, cin, c, s if i == 0 else 1))
            cin = c
    split = [4, 7, 11, 17]
    if alphas is None:
        key = "mobilenetv2_ee" if (in_hw, n_classes, seed) == (224, 1000, 2) else None
        alphas = load_calibration().get(key, {}).get("alphas", [6.0] * 4) if key else [6.0] * 4
    stages = []
    b0 = 0
    for s, b1 in enumerate(split):
        rng = _rng(seed, 300 + s)
        layers: List[Layer] = []
        idx = FROM_STAGE_INPUT
        if s == 0:
            layers.append(_conv(rng, OP_CONV, 3, 32, 3, 2, 1, ACT_RELU6, bf16=bf16))
            idx = 0
        for (t, ci, co, st) in blocks[b0:b1]:
            hid = ci * t
            src = idx
            if t != 1:
                layers.append(_conv(rng, OP_CONV, ci, hid, 1, 1, 0, ACT_RELU6, bf16=bf16, input_from=src))
                dw_in = len(layers) - 1
            else:
                dw_in = src
            layers.append(_conv(rng, OP_DWCONV, hid, hid, 3, st, 1, ACT_RELU6, bf16=bf16, input_from=dw_in))
            res = src if (st == 1 and ci == co) else NO_RESIDUAL
            layers.append(_conv(rng, OP_CONV, hid, co, 1, 1, 0, ACT_NONE, gamma=0.7, bf16=bf16, residual_from=res))
            idx = len(layers) - 1
        c_out = blocks[b1 - 1][2]
        last = s == len(split) - 1
        if last:
            layers.append(_conv(rng, OP_CONV, c_out, 1280, 1, 1, 0, ACT_RELU6, bf16=bf16))
            c_out = 1280
        fw, fb = head_weights(seed, 300 + s, c_out, n_classes, alphas[s], bf16)
        stages.append(Stage(layers, n_classes, fw, fb, 1.0 if last else threshold, last))
        b0 = b1
    return Model("mobilenetv2_ee", dtype, in_hw, in_hw, 3, stages, max_batch,
                 {"seed": seed, "alphas": list(alphas), "threshold": threshold})


def benchmark_model(workload: str, max_batch: int, flat_heads: bool = False):
    """The benchmark configurations by name: (model, input seed).  ``flat_heads`` scales the FC weights down so that
    unshifted confidences sit near 1/n_classes and only forced logit shifts (exit-rate sweep) decide who leaves."""
    if workload == "resnet50":
        return resnet50_ee(seed=1, max_batch=max_batch, alphas=[0.01] * 4 if flat_heads else None), 1
    if workload == "mobilenetv2":
        return mobilenetv2_ee(seed=2, max_batch=max_batch, alphas=[0.01] * 4 if flat_heads else None), 2
    if workload == "tiny":
        return tiny_ee_cnn(seed=0, max_batch=max_batch), 0
    raise ValueError(f"unknown workload {workload}")


def factorised_tower_ee(seed: int = 5, max_batch: int = 32, in_hw: int = 68, width: int = 192, n_classes: int = 1000,
                        blocks=(2, 2), dtype: str = "bf16", alphas=None, threshold: float = 0.6) -> Model:
    """A backbone in the shape of the 17 x 17 towers of Inception-v3 (the paper's second benchmark network, Section IV):
    a strided 3x3 stem pair brings the image to in_hw / 4, then every stage is a run of residual blocks
    1x1 -> 1x7 -> 7x1 -> 1x1 (+ block input), the 1 x 7 and 7 x 1 filters padded only along their own axis.  The
    branches of the original (concatenated towers, pooled branch) are not modelled: this workload exists for the
    asymmetric filters.  Exit heads (GAP + FC) after every stage, the last one always taken."""
    bf16 = dtype == "bf16"
    alphas = alphas or [6.0] * len(blocks)
    stages = []
    cin = 3
    for s, nb in enumerate(blocks):
        rng = _rng(seed, 400 + s)
        layers: List[Layer] = []
        idx = FROM_STAGE_INPUT
        if s == 0:
            layers.append(_conv(rng, OP_CONV, 3, 32, 3, 2, 1, ACT_RELU, bf16=bf16))
            layers.append(_conv(rng, OP_CONV, 32, width, 3, 2, 1, ACT_RELU, bf16=bf16))
            idx, cin = 1, width
        elif cin != width << s:
            layers.append(_conv(rng, OP_CONV, cin, width << s, 1, 2, 0, ACT_RELU, bf16=bf16, input_from=idx))
            idx, cin = len(layers) - 1, width << s
        mid = cin // 2
        for _ in range(nb):
            layers.append(_conv_hw(rng, cin, mid, 1, 1, 1, 0, 0, ACT_RELU, bf16=bf16, input_from=idx))
            layers.append(_conv_hw(rng, mid, mid, 1, 7, 1, 0, 3, ACT_RELU, bf16=bf16))
            layers.append(_conv_hw(rng, mid, mid, 7, 1, 1, 3, 0, ACT_RELU, bf16=bf16))
            layers.append(_conv_hw(rng, mid, cin, 1, 1, 1, 0, 0, ACT_RELU, gamma=0.3, bf16=bf16, residual_from=idx))
            idx = len(layers) - 1
        last = s == len(blocks) - 1
        fw, fb = head_weights(seed, 400 + s, cin, n_classes, alphas[s], bf16)
        stages.append(Stage(layers, n_classes, fw, fb, 1.0 if last else threshold, last))
    return Model("factorised_tower_ee", dtype, in_hw, in_hw, 3, stages, max_batch, {"seed": seed})


# ----------------------------------------------------------------------------- inputs

def make_input(model: Model, batch: int, seed: int, first_id: int = 0, rho: float = 0.5, grid: int = 4) -> np.ndarray:
    """Images whose every pixel is marginally N(0,1), NHWC.

    ``x = sqrt(1-rho) * white + sqrt(rho) * coarse`` where ``white`` is i.i.d. N(0,1) per
    element and ``coarse`` is an i.i.d. N(0,1) field on a ``grid x grid`` lattice per channel,
    repeated over blocks of pixels.  The coarse part gives every sample its own global
    structure; with white noise alone the global-average-pool of a random-init network is
    almost the same vector for every sample and all confidences coincide.

    Sample ``i`` depends only on (seed, first_id + i): the same id gives the same image in
    any batch, which is what the batch-invariance tests rely on."""
    H, W, Cc = model.in_h, model.in_w, model.in_c
    x = np.empty((batch, H, W, Cc), dtype=np.float32)
    a, b = np.float32(np.sqrt(1.0 - rho)), np.float32(np.sqrt(rho))
    for i in range(batch):
        g = _rng(seed, 7, first_id + i)
        white = g.standard_normal((H, W, Cc), dtype=np.float32)
        coarse = g.standard_normal((grid, grid, Cc), dtype=np.float32)
        coarse = np.repeat(np.repeat(coarse, -(-H // grid), axis=0), -(-W // grid), axis=1)[:H, :W]
        x[i] = a * white + b * coarse
    return to_bf16_grid(x) if model.dtype == "bf16" else x


def random_features(shape, seed: int, bf16: bool, relu: bool = True) -> np.ndarray:
    """Stand-in stage-boundary features (non-negative like a post-ReLU map when ``relu``)."""
    x = _rng(seed, 11).standard_normal(shape, dtype=np.float32)
    if relu:
        x = np.abs(x)
    return to_bf16_grid(x) if bf16 else x


def bernoulli_exit_shifts(seed: int, n_ids: int, n_exits: int, p: float, n_classes: int, shift: float = 16.0):
    """Config-4 forcing: for every (sample id, exit) one seeded Bernoulli(p) draw; a drawn
    sample gets ``shift`` added to logit ``id mod n_classes`` at that exit.  Returns
    (draws uint8 [n_exits][n_ids], shift float32 [n_exits][n_ids], cls int32 [n_ids])."""
    u = _rng(seed, 13).random((n_exits, n_ids))
    draws = (u < p).astype(np.uint8)
    cls = (np.arange(n_ids) % n_classes).astype(np.int32)
    return draws, (draws * np.float32(shift)).astype(np.float32), cls


def poisson_arrivals(seed: int, n: int, rate_per_s: float) -> np.ndarray:
    """Arrival times (seconds) of ``n`` requests with exponential inter-arrival gaps
    (Section IV: arrival times follow a Poisson process at the stated rate)."""
    gaps = _rng(seed, 17).exponential(1.0 / rate_per_s, size=n)
    return np.cumsum(gaps)
