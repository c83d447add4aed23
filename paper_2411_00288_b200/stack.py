"""Run a stack of convolutions (synth.StackStep) through the library, layer by layer.

Only marshalling: weights are masked and compressed once with the library's own calls, output
buffers are allocated once, and forward() issues one C-ABI call per convolution on the current
stream (so it can be recorded into a CUDA graph); the 3x3 stride-2 max-pool between the stem and
the first block is the library's ssconv_maxpool.  A dense layer with 8 input channels (the stem) runs
as ssconv_unfold_w followed by the equivalent KH x 1 convolution over the unfolded taps.
"""
from __future__ import annotations

from typing import List, Optional

import torch

from . import api, synth


class ConvStack:
    def __init__(self, steps: List[synth.StackStep], device, with_dense: bool = False):
        self.steps = steps
        self.device = torch.device(device)
        self.layers = []
        self.outputs: List[Optional[torch.Tensor]] = []
        self.status = torch.zeros(1, dtype=torch.int32, device=self.device)
        shape = None
        shapes = []
        for st in steps:
            if st.kind == "maxpool":
                n, h, w, c = shapes[st.src]
                shape = (n, (h + 2 - 3) // 2 + 1, (w + 2 - 3) // 2 + 1, c)
                self.layers.append(None)
            else:
                spec = st.spec
                inp = synth.make_weights(spec)
                desc = api.desc_from_spec(spec)
                w = inp.w.to(self.device)
                bias = inp.bias.to(self.device) if inp.bias is not None else None
                entry = dict(desc=desc, w=None, bias=bias, w_comp=None, meta=None, w_host=inp.w, bias_host=inp.bias)
                if st.kind == "conv":
                    pat = api.ssconv_select_mask(api.MASK_MAGNITUDE_BF16, w, spec.G)
                    entry["w_comp"], entry["meta"] = api.ssconv_compress(desc, w, pat)
                    entry["pattern"] = pat
                if st.kind == "dense" or with_dense:
                    entry["w"] = w
                if st.kind == "dense" and spec.C_in == 8 and spec.KW > 1:
                    # the filter row's taps as channels: x -> [N,H,W_out,C_pad], weights -> [C_out,KH,1,C_pad]
                    c_pad = -(-spec.KW * spec.C_in // 64) * 64
                    entry["unfold"] = dict(
                        c_pad=c_pad, w=api.ssconv_unfold_w(w, spec.KW, C_pad=c_pad),
                        x=torch.empty((spec.N, spec.H, spec.W_out, c_pad), dtype=torch.bfloat16, device=self.device),
                        desc=api.make_desc(spec.N, spec.H, spec.W_out, c_pad, spec.C_out, spec.KH, 1,
                                           stride=(spec.stride, 1), pad=(spec.pad, 0), dil=(spec.dil, 1),
                                           bias=spec.has_bias, relu=spec.relu and not spec.gelu, gelu=spec.gelu))
                self.layers.append(entry)
                shape = (spec.N, spec.H_out, spec.W_out, spec.C_out)
            shapes.append(shape)
            self.outputs.append(torch.empty(shape, dtype=torch.bfloat16, device=self.device))
        torch.cuda.synchronize(self.device)

    def forward(self, x: torch.Tensor, sparse: bool = True) -> torch.Tensor:
        """Enqueue the whole stack; returns the last chained output (not synchronised)."""
        last = None
        for i, st in enumerate(self.steps):
            src = x if st.src < 0 else self.outputs[st.src]
            y = self.outputs[i]
            if st.kind == "maxpool":
                api.ssconv_maxpool(src, 3, 2, 1, y=y)
            else:
                L = self.layers[i]
                res = self.outputs[st.res] if st.res >= 0 else None
                if st.kind == "conv" and sparse:
                    api.ssconv_forward(L["desc"], src, L["w_comp"], L["meta"], L["bias"], y=y, dev_status=self.status,
                                       residual=res)
                elif "unfold" in L:
                    U = L["unfold"]
                    sp = st.spec
                    api.ssconv_unfold_w(src, sp.KW, sp.stride, sp.pad, sp.dil, C_pad=U["c_pad"], y=U["x"])
                    api.ssconv_forward_dense(U["desc"], U["x"], U["w"], L["bias"], y=y, dev_status=self.status,
                                             residual=res)
                else:
                    api.ssconv_forward_dense(L["desc"], src, L["w"], L["bias"], y=y, dev_status=self.status,
                                             residual=res)
            if st.feeds_next:
                last = y
        return last

    def conv_flops(self) -> int:
        return sum(st.spec.dense_equiv_flops for st in self.steps if st.kind != "maxpool")
