"""Run a stack of convolutions (synth.StackStep) through the library, layer by layer.

Only marshalling: weights are masked and compressed once with the library's own calls, output
buffers are allocated once, and forward() issues one C-ABI call per convolution on the current
stream (so it can be recorded into a CUDA graph); the 3x3 stride-2 max-pool between the stem and
the first block is the library's ssconv_maxpool.  The stem (a dense strided convolution over very few
channels) has two forms, chosen by the channel count of the tensor handed to forward(): raw images
(fewer channels than the stem's padded C_in, e.g. RGB) go through ssconv_space_to_depth and the
equivalent T x 1 convolution on a sliding-window view (ssconv_forward_dense_strided); images already
padded to the stem's C_in go through ssconv_unfold_w and the equivalent KH x 1 convolution.
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
                shape = (n, api.ssconv_window_extent(h, 3, 2, 1), api.ssconv_window_extent(w, 3, 2, 1), c)
                self.layers.append(None)
            else:
                spec = st.spec
                inp = synth.make_weights(spec)
                desc = api.desc_from_spec(spec)
                w = inp.w.to(self.device)
                bias = inp.bias.to(self.device) if inp.bias is not None else None
                entry = dict(desc=desc, w=None, bias=bias, w_comp=None, meta=None, w_host=inp.w, bias_host=inp.bias)
                fold = api.ssconv_fold_factor(desc) if st.kind == "conv" else 1
                entry["fold"] = fold
                if st.kind == "conv":
                    pat = api.ssconv_select_mask(api.MASK_MAGNITUDE_BF16, w, spec.G)
                    entry["pattern"] = pat
                    if fold > 1:
                        # neighbouring output pixels as extra output channels: weights, patterns and bias are
                        # rearranged once, the layer then runs under the folded descriptor on the same bytes
                        entry["desc"] = api.ssconv_fold_desc(desc, fold)
                        w_f, entry["bias"] = api.ssconv_fold_weights(desc, fold, w, bias)
                        pat_f, _ = api.ssconv_fold_weights(desc, fold, pat)
                        entry["w_comp"], entry["meta"] = api.ssconv_compress(entry["desc"], w_f, pat_f)
                        w = w_f
                    else:
                        entry["w_comp"], entry["meta"] = api.ssconv_compress(desc, w, pat)
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
                if st.kind == "dense" and spec.C_in == 8 and spec.KH == spec.KW and spec.stride > 1 and st.src < 0:
                    entry["s2d"] = self._prepare_s2d(spec, w, real_c=3, bias=bias)
                self.layers.append(entry)
                shape = (spec.N, spec.H_out, spec.W_out, spec.C_out)
            shapes.append(shape)
            self.outputs.append(torch.empty(shape, dtype=torch.bfloat16, device=self.device))
        torch.cuda.synchronize(self.device)

    def _prepare_s2d(self, spec, w: torch.Tensor, real_c: int, bias: Optional[torch.Tensor]):
        """Buffers, weights and descriptor of the space-to-depth form of a K x K stride-s layer on images
        of `real_c` channels: blocks of s x s pixels become one pixel of C_pad channels, and the layer is a
        T x T convolution of unit stride without padding over them, T = ceil(K/s).  With few output
        channels two output pixels of a row are folded into the output channels (T + 1 taps of stride 2
        along the width); the taps of a row are then read as one pixel of 64 channels through a sliding
        window over neighbouring block pixels, which leaves a T x 1 convolution for the tensor cores."""
        s, K = spec.stride, spec.KH
        T = -(-K // s)
        c_blk = s * s * real_c
        c_pad = -(-c_blk // 4) * 4
        w_real = w[..., :real_c].contiguous()
        w_s2d = api.ssconv_space_to_depth(w_real, s, 0, T, T, c_pad)          # [C_out, T, T, c_pad]
        hb, wb = spec.H_out + T - 1, spec.W_out + T - 1
        conv = api.make_desc(spec.N, hb, wb, c_pad, spec.C_out, T, T, stride=1, pad=0, dil=1)
        f = 2 if (2 * spec.C_out <= 128 and spec.W_out % 2 == 0 and (T + 1) * c_pad <= 64 and (2 * c_pad) % 8 == 0) else 1
        taps = T + f - 1
        c_view = -(-taps * c_pad // 64) * 64
        wb += wb % 2                                                            # row pitch a multiple of 16 bytes
        w_f, bias_f = api.ssconv_fold_weights(conv, f, w_s2d, bias)            # [f C_out, T, taps, c_pad]
        w_view = api.ssconv_pad_channels(w_f.view(-1, taps * c_pad), C_pad=c_view).view(f * spec.C_out, T, 1, c_view)
        desc = api.make_desc(spec.N, hb, spec.W_out // f, c_view, f * spec.C_out, T, 1, stride=1, pad=0, dil=1,
                             bias=spec.has_bias, relu=spec.relu and not spec.gelu, gelu=spec.gelu)
        # the window of the last pixel of the last row ends c_view - taps*c_pad channels past the buffer's rows
        slack = c_view
        buf = torch.zeros((spec.N * hb * wb * c_pad + slack,), dtype=torch.bfloat16, device=self.device)
        return dict(block=s, pad=spec.pad, hb=hb, wb=wb, c_pad=c_pad, real_c=real_c, w=w_view, bias=bias_f, desc=desc,
                    fold=f, strides=(f * c_pad, wb * c_pad, hb * wb * c_pad),
                    x=buf[:spec.N * hb * wb * c_pad].view(spec.N, hb, wb, c_pad))

    def run_step(self, i: int, x: torch.Tensor, sparse: bool = True) -> torch.Tensor:
        """Enqueue step i alone (its input must already be in place); returns its output tensor."""
        st = self.steps[i]
        src = x if st.src < 0 else self.outputs[st.src]
        y = self.outputs[i]
        if st.kind == "maxpool":
            api.ssconv_maxpool(src, 3, 2, 1, y=y)
            return y
        L = self.layers[i]
        res = self.outputs[st.res] if st.res >= 0 else None
        if st.kind == "conv" and sparse:
            api.ssconv_forward(L["desc"], src, L["w_comp"], L["meta"], L["bias"], y=y, dev_status=self.status,
                               residual=res)
        elif "s2d" in L and src.shape[-1] == L["s2d"]["real_c"]:
            S = L["s2d"]
            api.ssconv_space_to_depth(src, S["block"], S["pad"], S["hb"], S["wb"], S["c_pad"], y=S["x"])
            api.ssconv_forward_dense_strided(S["desc"], S["x"], S["strides"], S["w"], S["bias"], y=y,
                                             dev_status=self.status)
        elif "unfold" in L:
            U = L["unfold"]
            sp = st.spec
            api.ssconv_unfold_w(src, sp.KW, sp.stride, sp.pad, sp.dil, C_pad=U["c_pad"], y=U["x"])
            api.ssconv_forward_dense(U["desc"], U["x"], U["w"], L["bias"], y=y, dev_status=self.status, residual=res)
        else:
            api.ssconv_forward_dense(L["desc"], src, L["w"], L["bias"], y=y, dev_status=self.status, residual=res)
        return y

    def forward(self, x: torch.Tensor, sparse: bool = True) -> torch.Tensor:
        """Enqueue the whole stack; returns the last chained output (not synchronised)."""
        last = None
        for i, st in enumerate(self.steps):
            y = self.run_step(i, x, sparse)
            if st.feeds_next:
                last = y
        return last

    def conv_flops(self) -> int:
        return sum(st.spec.dense_equiv_flops for st in self.steps if st.kind != "maxpool")
