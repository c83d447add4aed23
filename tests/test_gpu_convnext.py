"""A ConvNeXt-T-shaped network chained through the library, every step against its oracle.

Teacher-forced like the ResNet stack: each step's oracle receives the bf16 input the GPU step before it
actually produced, so each step meets the gates of a stand-alone call.  The stem is checked as the 4x4
stride-4 convolution on the RGB image it stands for (the space-to-depth form is the library's business)."""
import numpy as np
import pytest
import torch

from oracle import blocks, masks
from oracle.conv import ConvShape, conv2d_f64, conv2d_f64_sample
from paper_2411_00288_b200 import api, convnext, synth
from tests import parity

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _check(net, x, sample):
    worst = ("", 0.0, 0.0)
    peak, peak_step = 0.0, ""
    for i, st in enumerate(net.steps):
        P = net.params[i]
        y = net.outputs[i].cpu()
        src = x if st.src < 0 else net.outputs[st.src].cpu()
        yg_full = parity.bf16_tensor_to_f64(y)
        if float(np.abs(yg_full).max()) > peak:
            peak, peak_step = float(np.abs(yg_full).max()), st.name
        if st.kind == "s2d":
            continue          # checked through the stem convolution below (and bit-exact in its own test)
        if st.kind == "layernorm":
            ref = blocks.layernorm_f64(parity.bf16_tensor_to_f64(src), P["gamma_host"].numpy(), P["beta_host"].numpy(),
                                       convnext.LN_EPS)
            err = np.abs(yg_full - ref)
            assert (err <= 2.0 ** -8 * np.abs(ref) + 1e-3).all(), (st.name, err.max())
            continue
        d = st.desc
        if st.kind == "depthwise":
            shp = ConvShape(d.N, d.H, d.W, d.C_in, d.C_out, d.KH, d.KW, (1, 1), (d.pad_h, d.pad_w), (1, 1), relu=False)
            ref = blocks.depthwise_conv2d_f64(shp, synth.bf16_bits(src), synth.bf16_bits(P["w_host"]),
                                              bias=P["bias_host"].numpy())
            rel, mx = parity.errors(yg_full, ref)
        else:
            if st.name == "stem_conv":   # the convolution the stem stands for, on the raw images
                shp = ConvShape(d.N, x.shape[1], x.shape[2], 3, d.C_out, 4, 4, (4, 4), (0, 0), (1, 1), relu=False)
                src_bits, w_bits, mask = synth.bf16_bits(x), synth.bf16_bits(P["w_host"]), None
            else:
                shp = ConvShape(d.N, d.H, d.W, d.C_in, d.C_out, d.KH, d.KW, (d.stride_h, d.stride_w), (d.pad_h, d.pad_w),
                                (1, 1), relu=False)
                src_bits, w_bits = synth.bf16_bits(src), synth.bf16_bits(P["w_host"])
                pat = masks.select_from_magnitude(w_bits)
                assert np.array_equal(pat, P["pattern"].cpu().numpy()), st.name
                mask = masks.mask_from_pattern(pat, w_bits.shape)
            res = net.outputs[st.res].cpu() if st.res >= 0 else None
            if sample is None:
                ref = conv2d_f64(shp, src_bits, w_bits, mask=mask, bias=P["bias_host"].numpy())
                if res is not None:
                    ref = ref + parity.bf16_tensor_to_f64(res)
                yg = yg_full
            else:
                rng = np.random.default_rng(1000 + i)
                idx = rng.choice(y.numel(), size=min(sample, y.numel()), replace=False)
                ref = conv2d_f64_sample(shp, src_bits, w_bits, idx, mask=mask, bias=P["bias_host"].numpy())
                if res is not None:
                    ref = ref + parity.bf16_tensor_to_f64(res).reshape(-1)[idx]
                yg = yg_full.reshape(-1)[idx]
            if st.gelu:
                ref = parity.gelu_f64(ref)
            rel, mx = parity.errors(yg, ref)
        assert rel <= parity.REL_FRO_TOL and mx <= parity.MAX_ABS_TOL, f"{st.name}: rel={rel:.3e} max={mx:.3e}"
        if rel > worst[1]:
            worst = (st.name, rel, mx)
    print("worst step", worst, "largest |activation|", peak, "in", peak_step)
    assert peak < 16.0, peak_step     # (the gates above hold; bf16 rounds to 2^-5 from 8 up, which they could not absorb for long)


def _images(n, image):
    g = torch.Generator().manual_seed(synth.SEED_BASE + 6100 + n)
    return torch.randn((n, image, image, 3), generator=g, dtype=torch.float32).to(torch.bfloat16)


def test_convnext_t_batch2_every_step_full():
    net = convnext.ConvNeXtStack(2, DEV)
    x = _images(2, 224)
    net.forward(x.to(DEV))
    torch.cuda.synchronize()
    assert int(net.status.item()) == 0
    assert len(net.steps) == 3 + 18 * 4 + 3 * 2
    _check(net, x, None)


def test_convnext_t_batch32_sampled_and_the_dense_counterpart_agrees():
    net = convnext.ConvNeXtStack(32, DEV)
    x = _images(32, 224)
    out = net.forward(x.to(DEV)).clone()
    torch.cuda.synchronize()
    assert int(net.status.item()) == 0
    _check(net, x, 32768)
    assert tuple(out.shape) == (32, 7, 7, 768)
