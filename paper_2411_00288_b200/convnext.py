"""A ConvNeXt-T-shaped network run through the library, step by step.

Only marshalling, like stack.py: seeded synthetic weights (no trained ones exist here), masks by
magnitude selected and compressed once with the library's own calls, buffers allocated once, and
forward() issuing one C-ABI call per step on the current stream (so it can be recorded into a CUDA
graph).  The paper masks the dense convolutions of the ConvNeXts it evaluates and leaves the grouped
(depthwise) ones untouched (Sec. 4); here that means

  stem        4x4 stride-4 convolution 3 -> 96 on the RGB image (dense: 3 input channels), run as
              space-to-depth (blocks of 4 x 4 pixels = 48 channels) + a 1x1 convolution; layer norm
  block       depthwise 7x7 (dense) -> layer norm -> 1x1 C -> 4C (2:4 masked, GELU)
              -> 1x1 4C -> C (2:4 masked, the layer scale folded into weights and bias, skip connection fused)
  downsample  layer norm -> 2x2 stride-2 convolution C -> 2C (2:4 masked)

with depths (3, 3, 9, 3) and widths (96, 192, 384, 768).  Every step keeps its output, so a test can
check each one against its oracle on the input the step before actually produced.
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import List, Optional

import torch

from . import api, synth

DEPTHS = (3, 3, 9, 3)
WIDTHS = (96, 192, 384, 768)
LAYER_SCALE = 0.3      # folded into the second point-wise convolution of a block
LN_EPS = 1e-6


@dataclass
class Step:
    kind: str                 # "s2d", "dense", "conv", "depthwise", "layernorm"
    name: str
    src: int                  # index of the step whose output it reads (-1: the images)
    res: int = -2             # index of the step whose output is added (fused skip connection)
    desc: Optional[api.Desc] = None
    gelu: bool = False


class ConvNeXtStack:
    def __init__(self, batch: int, device, image: int = 224, depths=DEPTHS, widths=WIDTHS, seed: int = 0):
        self.device = torch.device(device)
        self.batch = batch
        self.steps: List[Step] = []
        self.params: List[dict] = []
        self.outputs: List[torch.Tensor] = []
        self.status = torch.zeros(1, dtype=torch.int32, device=self.device)
        self.g = torch.Generator().manual_seed(synth.SEED_BASE + 6000 + seed)
        dev = self.device
        n = batch
        hw = image // 4
        c0 = widths[0]
        # ---- stem
        self._add(Step("s2d", "stem_s2d", -1), dict(block=4, c_pad=48), (n, hw, hw, 48))
        w_stem = self._randn((c0, 4, 4, 3), (2.0 / 48) ** 0.5)
        b_stem = self._bias(c0)
        w_s2d = api.ssconv_space_to_depth(w_stem.to(dev), 4, 0, 1, 1, 48)          # [C, 1, 1, 48]
        d = api.make_desc(n, hw, hw, 48, c0, 1, 1, bias=True)
        self._add(Step("dense", "stem_conv", 0, desc=d), dict(w=w_s2d, bias=b_stem.to(dev), w_host=w_stem, bias_host=b_stem),
                  (n, hw, hw, c0))
        self._ln("stem_ln", len(self.steps) - 1, c0, (n, hw, hw, c0))
        src = len(self.steps) - 1
        c = c0
        for stage, (depth, width) in enumerate(zip(depths, widths)):
            if stage > 0:
                self._ln(f"s{stage}_down_ln", src, c, (n, hw, hw, c))
                hw //= 2
                d = api.make_desc(n, 2 * hw, 2 * hw, c, width, 2, 2, stride=2, pad=0, bias=True)
                self._conv(f"s{stage}_down", len(self.steps) - 1, d, (n, hw, hw, width), scale=1.0)
                src = len(self.steps) - 1
                c = width
            for b in range(depth):
                tag = f"s{stage}b{b}"
                block_in = src
                d_dw = api.make_desc(n, hw, hw, c, c, 7, 7, 1, 3, bias=True)
                w_dw = self._randn((7, 7, c), 0.1)
                b_dw = self._bias(c)
                self._add(Step("depthwise", tag + "_dw", block_in, desc=d_dw),
                          dict(w=w_dw.to(dev), bias=b_dw.to(dev), w_host=w_dw, bias_host=b_dw), (n, hw, hw, c))
                self._ln(tag + "_ln", len(self.steps) - 1, c, (n, hw, hw, c))
                d1 = api.make_desc(n, hw, hw, c, 4 * c, 1, 1, bias=True, gelu=True)
                self._conv(tag + "_pw1", len(self.steps) - 1, d1, (n, hw, hw, 4 * c), scale=1.0, gelu=True)
                d2 = api.make_desc(n, hw, hw, 4 * c, c, 1, 1, bias=True)
                self._conv(tag + "_pw2", len(self.steps) - 1, d2, (n, hw, hw, c), scale=LAYER_SCALE, res=block_in)
                src = len(self.steps) - 1
        torch.cuda.synchronize(self.device)

    # ---- construction helpers
    def _randn(self, shape, std):
        return (torch.randn(shape, generator=self.g, dtype=torch.float32) * std).to(torch.bfloat16)

    def _bias(self, c, std=0.1):
        return torch.randn((c,), generator=self.g, dtype=torch.float32) * std

    def _add(self, step: Step, params: dict, shape):
        self.steps.append(step)
        self.params.append(params)
        self.outputs.append(torch.empty(shape, dtype=torch.bfloat16, device=self.device))

    def _ln(self, name, src, c, shape):
        gamma = 1.0 + 0.1 * torch.randn((c,), generator=self.g, dtype=torch.float32)
        beta = 0.1 * torch.randn((c,), generator=self.g, dtype=torch.float32)
        self._add(Step("layernorm", name, src), dict(gamma=gamma.to(self.device), beta=beta.to(self.device),
                                                      gamma_host=gamma, beta_host=beta), shape)

    def _conv(self, name, src, desc, shape, scale, gelu=False, res=-2):
        k = desc.KH * desc.KW * desc.C_in
        w = self._randn((desc.C_out, desc.KH, desc.KW, desc.C_in), scale / k ** 0.5)
        bias = self._bias(desc.C_out, 0.1 * scale)
        wd = w.to(self.device)
        pat = api.ssconv_select_mask(api.MASK_MAGNITUDE_BF16, wd, wd.numel() // 4)
        w_comp, meta = api.ssconv_compress(desc, wd, pat)
        self._add(Step("conv", name, src, res=res, desc=desc, gelu=gelu),
                  dict(w=wd, w_comp=w_comp, meta=meta, bias=bias.to(self.device), pattern=pat, w_host=w, bias_host=bias), shape)

    # ---- execution
    def run_step(self, i: int, x: torch.Tensor, sparse: bool = True) -> torch.Tensor:
        st, P, y = self.steps[i], self.params[i], self.outputs[i]
        src = x if st.src < 0 else self.outputs[st.src]
        if st.kind == "s2d":
            api.ssconv_space_to_depth(src, P["block"], 0, y.shape[1], y.shape[2], P["c_pad"], y=y)
        elif st.kind == "dense":
            api.ssconv_forward_dense(st.desc, src, P["w"], P["bias"], y=y, dev_status=self.status)
        elif st.kind == "depthwise":
            api.ssconv_depthwise(st.desc, src, P["w"], P["bias"], y=y)
        elif st.kind == "layernorm":
            api.ssconv_layernorm(src, P["gamma"], P["beta"], LN_EPS, y=y)
        else:
            res = self.outputs[st.res] if st.res >= 0 else None
            if sparse:
                api.ssconv_forward(st.desc, src, P["w_comp"], P["meta"], P["bias"], y=y, dev_status=self.status,
                                   residual=res)
            else:
                api.ssconv_forward_dense(st.desc, src, P["w"], P["bias"], y=y, dev_status=self.status, residual=res)
        return y

    def forward(self, x: torch.Tensor, sparse: bool = True) -> torch.Tensor:
        """Enqueue the whole network on images x [N, H, W, 3] bf16; returns the last feature map (not synchronised)."""
        y = None
        for i in range(len(self.steps)):
            y = self.run_step(i, x, sparse)
        return y

    def masked_conv_flops(self) -> int:
        total = 0
        for st, y in zip(self.steps, self.outputs):
            if st.kind == "conv":
                d = st.desc
                total += 2 * y.shape[0] * y.shape[1] * y.shape[2] * d.C_out * d.KH * d.KW * d.C_in
        return total
