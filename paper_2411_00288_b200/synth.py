"""Seeded synthetic inputs and layer shapes for the 2:4 masked convolution workloads.

This module only draws random tensors and lists layer shapes; it contains none of the
method's arithmetic (no mask selection, no convolution) and imports neither the CUDA
binding nor the CPU oracle, so both sides of a parity test can be fed the same bits.

The tensors stand in for ImageNet-normalised activations and pretrained Torchvision
weights, neither of which is available offline: activations are N(0,1), weights are
zero-mean normal with a fan-in scaled deviation so that outputs stay O(1).
"""
from __future__ import annotations

import math
from dataclasses import dataclass, replace
from typing import List, Optional

import numpy as np
import torch

SEED_BASE = 241100288 * 1000


@dataclass(frozen=True)
class LayerSpec:
    name: str
    N: int
    H: int
    W: int
    C_in: int
    C_out: int
    KH: int
    KW: int
    stride: int = 1
    pad: int = 0
    dil: int = 1
    relu: bool = True
    has_bias: bool = True
    gelu: bool = False             # GELU instead of ReLU (takes precedence)
    w_std: str = "fan_in"          # "fan_in": 1/sqrt(fan_in); "he": sqrt(2/fan_in); or a float as str
    mask_source: str = "magnitude"  # "magnitude" | "gumbel_logits" | "uniform_pattern"
    config: int = 0
    index: int = 0
    extra: bool = False            # parity-only row, not part of the timed sweep

    @property
    def K(self) -> int:
        return self.KH * self.KW * self.C_in

    @property
    def G(self) -> int:
        return self.C_out * self.K // 4

    @property
    def H_out(self) -> int:
        return (self.H + 2 * self.pad - self.dil * (self.KH - 1) - 1) // self.stride + 1

    @property
    def W_out(self) -> int:
        return (self.W + 2 * self.pad - self.dil * (self.KW - 1) - 1) // self.stride + 1

    @property
    def P(self) -> int:
        return self.N * self.H_out * self.W_out

    @property
    def seed(self) -> int:
        return SEED_BASE + 100 * self.config + self.index

    @property
    def dense_equiv_flops(self) -> int:
        return 2 * self.P * self.C_out * self.K

    def algorithmic_bytes(self, sparse: bool = True) -> int:
        """Bytes the layer must move once: touched input, weights (+metadata), output, bias."""
        if self.KH == 1 and self.KW == 1 and self.stride > 1:
            touched = self.N * self.H_out * self.W_out * self.C_in
        else:
            touched = self.N * self.H * self.W * self.C_in
        wbytes = self.C_out * self.K + self.C_out * self.K // 8 if sparse else 2 * self.C_out * self.K
        return 2 * touched + wbytes + 2 * self.P * self.C_out + (4 * self.C_out if self.has_bias else 0)


def _number(specs: List[LayerSpec], config: int) -> List[LayerSpec]:
    return [replace(s, config=config, index=i) for i, s in enumerate(specs)]


def config_layers(config: int, batch: Optional[int] = None) -> List[LayerSpec]:
    """Layer shapes of the five workload configurations (batch overridable for small runs)."""
    if config == 1:
        n = batch or 1
        return _number([LayerSpec("c1_3x3_64", n, 14, 14, 64, 64, 3, 3, 1, 1, w_std="0.05",
                                  mask_source="uniform_pattern")], 1)
    if config == 2:
        n = batch or 32
        L = []
        for hw, c in ((56, 64), (28, 128), (14, 256), (7, 512)):
            L.append(LayerSpec(f"r18_3x3_{c}_{hw}", n, hw, hw, c, c, 3, 3, 1, 1))
        for hw, c in ((56, 64), (28, 128), (14, 256)):
            L.append(LayerSpec(f"r18_3x3s2_{c}to{2 * c}_{hw}", n, hw, hw, c, 2 * c, 3, 3, 2, 1))
        for hw, c in ((56, 64), (28, 128), (14, 256)):
            L.append(LayerSpec(f"r18_1x1s2_{c}to{2 * c}_{hw}", n, hw, hw, c, 2 * c, 1, 1, 2, 0, relu=False,
                               extra=True))
        return _number(L, 2)
    if config == 3:
        n = batch or 64
        L = []
        for hw, w in ((56, 64), (28, 128), (14, 256), (7, 512)):
            kw = dict(w_std="he", mask_source="gumbel_logits")
            L.append(LayerSpec(f"r50_1x1_{4 * w}to{w}_{hw}", n, hw, hw, 4 * w, w, 1, 1, **kw))
            L.append(LayerSpec(f"r50_3x3_{w}_{hw}", n, hw, hw, w, w, 3, 3, 1, 1, **kw))
            L.append(LayerSpec(f"r50_1x1_{w}to{4 * w}_{hw}", n, hw, hw, w, 4 * w, 1, 1, **kw))
        return _number(L, 3)
    if config == 4:
        n = batch or 128
        L = []
        for hw, d in ((56, 96), (28, 192), (14, 384), (7, 768)):
            L.append(LayerSpec(f"cnx_1x1_{d}to{4 * d}_{hw}", n, hw, hw, d, 4 * d, 1, 1, relu=True))
            L.append(LayerSpec(f"cnx_1x1_{4 * d}to{d}_{hw}", n, hw, hw, 4 * d, d, 1, 1, relu=False))
        return _number(L, 4)
    if config == 5:
        n = batch or 256
        L = []
        kw = dict(w_std="he")
        hw = 56
        c_prev = 64
        for stage, (width, blocks) in enumerate(((64, 3), (128, 4), (256, 6), (512, 3))):
            for b in range(blocks):
                s = 2 if (b == 0 and stage > 0) else 1
                tag = f"s{stage + 1}b{b}"
                L.append(LayerSpec(f"r50_{tag}_reduce", n, hw, hw, c_prev, width, 1, 1, **kw))
                L.append(LayerSpec(f"r50_{tag}_3x3", n, hw, hw, width, width, 3, 3, s, 1, **kw))
                if b == 0:
                    L.append(LayerSpec(f"r50_{tag}_down", n, hw, hw, c_prev, 4 * width, 1, 1, s, 0,
                                       relu=False, **kw))
                hw = hw // s
                L.append(LayerSpec(f"r50_{tag}_expand", n, hw, hw, width, 4 * width, 1, 1, **kw))
                c_prev = 4 * width
        return _number(L, 5)
    raise ValueError(f"unknown config {config}")


@dataclass(frozen=True)
class StackStep:
    """One step of a convolution stack: `kind` is "conv" (masked), "dense" (unmasked convolution)
    or "maxpool" (3x3, stride 2, pad 1).  `src` is the index of the step whose output it reads (-1:
    the stack's input); `feeds_next` is False for branches whose output nothing consumes."""
    kind: str
    spec: Optional[LayerSpec]
    src: int
    feeds_next: bool = True
    res: int = -2  # index of the step whose output is added before the activation (-2: none)


def resnet50_stack(batch: int = 256, residual: bool = False) -> List[StackStep]:
    """The convolution stack of a Torchvision-shaped ResNet-50: stem (7x7 stride 2, dense, on an
    input padded from 3 to 8 channels), 3x3 stride-2 max-pool, then per bottleneck reduce -> 3x3 ->
    expand with bias and ReLU, the expand output feeding the next block.  Every convolution has
    exactly the shape, traffic and FLOPs of the network's; batch norm counts as folded into the bias.
    residual=False: a residual-free chain, the four downsample convolutions read their block's
    input and feed nothing.  residual=True: the network's skip connections: the expand convolution
    adds the block's input (the downsample convolution's output in the first block of a stage)
    before its ReLU; the expand and downsample weights are scaled down so that activations stay
    O(1) over the 16 blocks without batch-norm statistics."""
    steps: List[StackStep] = []
    stem = LayerSpec("r50_stem", batch, 224, 224, 8, 64, 7, 7, 2, 3, w_std="he", config=5, index=90)
    steps.append(StackStep("dense", stem, -1))
    steps.append(StackStep("maxpool", None, 0))
    src = 1
    specs = config_layers(5, batch)
    i = 0
    while i < len(specs):
        block_in = src
        reduce_, conv3 = specs[i], specs[i + 1]
        steps.append(StackStep("conv", reduce_, block_in))
        steps.append(StackStep("conv", conv3, len(steps) - 1))
        after3 = len(steps) - 1
        i += 2
        identity = block_in
        if specs[i].name.endswith("_down"):
            down = specs[i]
            if residual:
                down = replace(down, w_std=str(0.5 * math.sqrt(1.0 / down.K)))
            steps.append(StackStep("conv", down, block_in, feeds_next=False))
            identity = len(steps) - 1
            i += 1
        if residual:
            expand = replace(specs[i], w_std=str(0.25 * math.sqrt(2.0 / specs[i].K)))
            steps.append(StackStep("conv", expand, after3, res=identity))
        else:
            steps.append(StackStep("conv", specs[i], after3))
        src = len(steps) - 1
        i += 1
    return steps


def make_weights(spec: LayerSpec, seed: Optional[int] = None) -> "LayerInputs":
    """Weights and bias only (no activations are drawn): for layers whose input comes from the
    layer before.  Its own seed stream, so the bits differ from make_inputs' for the same spec."""
    g = torch.Generator().manual_seed((spec.seed if seed is None else seed) + 50_000_000)
    w = (torch.randn((spec.C_out, spec.KH, spec.KW, spec.C_in), generator=g, dtype=torch.float32)
         * _std(spec)).to(torch.bfloat16)
    bias = (torch.randn((spec.C_out,), generator=g, dtype=torch.float32) * 0.1) if spec.has_bias else None
    return LayerInputs(spec, None, w, bias, None, None)


def _std(spec: LayerSpec) -> float:
    fan_in = spec.K
    if spec.w_std == "fan_in":
        return 1.0 / math.sqrt(fan_in)
    if spec.w_std == "he":
        return math.sqrt(2.0 / fan_in)
    return float(spec.w_std)


def bf16_bits(t: torch.Tensor) -> np.ndarray:
    """uint16 view of a CPU bf16 tensor's bit patterns (no copy of values, no rounding)."""
    assert t.dtype == torch.bfloat16 and t.device.type == "cpu"
    return t.contiguous().view(torch.int16).numpy().view(np.uint16)


@dataclass
class LayerInputs:
    spec: LayerSpec
    x: torch.Tensor                 # bf16 [N,H,W,C_in]
    w: torch.Tensor                 # bf16 [C_out,KH,KW,C_in]
    bias: Optional[torch.Tensor]    # fp32 [C_out]
    scores: Optional[torch.Tensor]  # fp32 [G,6] pattern scores with Gumbel noise already added
    pattern: Optional[torch.Tensor]  # uint8 [G], only for mask_source == "uniform_pattern"


def make_inputs(spec: LayerSpec, seed: Optional[int] = None, x_only: bool = False) -> LayerInputs:
    """Draw the layer's tensors on the CPU from one seeded generator, fp32 then bf16 (RNE)."""
    g = torch.Generator().manual_seed(spec.seed if seed is None else seed)
    x = torch.randn((spec.N, spec.H, spec.W, spec.C_in), generator=g, dtype=torch.float32).to(torch.bfloat16)
    if x_only:
        return LayerInputs(spec, x, None, None, None, None)
    w = (torch.randn((spec.C_out, spec.KH, spec.KW, spec.C_in), generator=g, dtype=torch.float32)
         * _std(spec)).to(torch.bfloat16)
    bias = (torch.randn((spec.C_out,), generator=g, dtype=torch.float32) * 0.1) if spec.has_bias else None
    scores = None
    pattern = None
    if spec.mask_source == "gumbel_logits":
        base = torch.randn((spec.G, 6), generator=g, dtype=torch.float32)
        u = torch.rand((spec.G, 6), generator=g, dtype=torch.float64).clamp_(1e-12, 1.0 - 1e-12)
        gumbel = -torch.log(-torch.log(u))
        scores = (base.double() + gumbel).float()
    elif spec.mask_source == "uniform_pattern":
        pattern = torch.randint(0, 6, (spec.G,), generator=g, dtype=torch.int64).to(torch.uint8)
    return LayerInputs(spec, x, w, bias, scores, pattern)


@dataclass
class TrainInputs:
    logits: torch.Tensor   # fp32 [G,6]: the trainable choice weights (log pi up to a constant)
    noise: torch.Tensor    # fp32 [G,6]: one Gumbel(0,1) draw per logit (the method's randomness, drawn here)
    dy: torch.Tensor       # bf16 [N,H_out,W_out,C_out]: a stand-in for the loss gradient at the layer's output


def make_train_inputs(spec: LayerSpec, seed: Optional[int] = None) -> TrainInputs:
    """Seeded inputs of one mask-learning step for a layer (its own stream of the layer's seed).
    The upstream gradient is N(0, 1/P) so that weight gradients stay O(1)."""
    g = torch.Generator().manual_seed((spec.seed if seed is None else seed) + 70_000_000)
    logits = torch.randn((spec.G, 6), generator=g, dtype=torch.float32)
    u = torch.rand((spec.G, 6), generator=g, dtype=torch.float64).clamp_(1e-12, 1.0 - 1e-12)
    noise = (-torch.log(-torch.log(u))).float()
    dy = (torch.randn((spec.N, spec.H_out, spec.W_out, spec.C_out), generator=g, dtype=torch.float32)
          / math.sqrt(spec.P)).to(torch.bfloat16)
    return TrainInputs(logits, noise, dy)
