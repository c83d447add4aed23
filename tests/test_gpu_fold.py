"""Folding of neighbouring output pixels into the output channels: the rearranged weights bit-exact
against a numpy construction from the definition, the folded layer (sparse and dense) against the fp64
oracle of the ORIGINAL layer, and the 12-channel space-to-depth forms against a numpy gather."""
import numpy as np
import pytest
import torch

from oracle import masks
from oracle.conv import conv2d_f64
from paper_2411_00288_b200 import api, synth
from tests import parity

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _fold_numpy(w, f, s, d):
    Co, KH, KW, per = w.shape
    KWf = (f - 1) * s + (KW - 1) * d + 1
    out = np.zeros((f * Co, KH, KWf, per), dtype=w.dtype)
    for j in range(f):
        for kw in range(KW):
            out[j * Co:(j + 1) * Co, :, j * s + kw * d] = w[:, :, kw]
    return out


@pytest.mark.parametrize("Co,KH,KW,C,f,s,d", [(64, 3, 3, 64, 2, 1, 1), (24, 3, 3, 16, 4, 1, 1), (16, 1, 5, 8, 2, 2, 1),
                                              (8, 2, 3, 8, 3, 1, 2), (64, 4, 4, 12, 2, 1, 1)])
def test_fold_weights_is_bit_exact(Co, KH, KW, C, f, s, d):
    g = torch.Generator().manual_seed(synth.SEED_BASE + 3400 + Co + KW)
    w = torch.randn((Co, KH, KW, C), generator=g).to(torch.bfloat16)
    bias = torch.randn((Co,), generator=g)
    W = 2 * f * s * 3 + (KW - 1) * d + 1 - s      # W_out = 6 f (a multiple of f) without padding
    desc = api.make_desc(1, 8, W, C, Co, KH, KW, stride=(1, s), pad=0, dil=(1, d))
    folded = api.ssconv_fold_desc(desc, f)
    assert (folded.C_out, folded.KW, folded.stride_w, folded.dil_w) == (f * Co, (f - 1) * s + (KW - 1) * d + 1, f * s, 1)
    assert api.ssconv_out_shape(folded)[1] * f == api.ssconv_out_shape(desc)[1] if C % 8 == 0 else True
    w2, b2 = api.ssconv_fold_weights(desc, f, w.to(DEV), bias.to(DEV))
    torch.cuda.synchronize()
    np.testing.assert_array_equal(synth.bf16_bits(w2.cpu()), _fold_numpy(synth.bf16_bits(w), f, s, d))
    np.testing.assert_array_equal(b2.cpu().numpy(), np.tile(bias.numpy(), f))
    if C % 4 == 0:
        pat = torch.randint(0, 6, (Co * KH * KW * C // 4,), generator=g, dtype=torch.int64).to(torch.uint8)
        p2, _ = api.ssconv_fold_weights(desc, f, pat.to(DEV))
        want = _fold_numpy(pat.numpy().reshape(Co, KH, KW, C // 4), f, s, d).reshape(-1)
        np.testing.assert_array_equal(p2.cpu().numpy(), want)


def test_fold_rules():
    d = api.make_desc(2, 56, 56, 64, 64, 3, 3, 1, 1)
    assert api.ssconv_fold_factor(d) == 2
    assert api.ssconv_fold_factor(api.make_desc(2, 56, 56, 64, 128, 3, 3, 1, 1)) == 1       # the rows are full already
    assert api.ssconv_fold_factor(api.make_desc(2, 56, 56, 256, 64, 1, 1, 1, 0)) == 1       # nothing to share between taps
    assert api.ssconv_fold_factor(api.make_desc(2, 55, 55, 64, 64, 3, 3, 1, 1)) == 1        # odd width
    with pytest.raises(api.SsconvError):
        api.ssconv_fold_desc(api.make_desc(2, 55, 55, 64, 64, 3, 3, 1, 1), 2)


CASES = [  # name, N, H, W, C_in, C_out, K, stride, pad, dil, f
    ("c64_3x3", 2, 14, 16, 64, 64, 3, 1, 1, 1, 2),
    ("c64_3x3_gelu_res", 2, 10, 12, 64, 64, 3, 1, 1, 1, 2),
    ("c32_3x3_f4", 2, 9, 16, 32, 32, 3, 1, 1, 1, 4),
    ("c64_3x3_s2", 2, 15, 15, 64, 48, 3, 2, 1, 1, 2),
    ("c40_5x5_dil2", 1, 12, 14, 16, 40, 5, 1, 4, 2, 2),
]


@pytest.mark.parametrize("case", CASES, ids=[c[0] for c in CASES])
@pytest.mark.parametrize("sparse", [True, False], ids=["sparse", "dense"])
def test_folded_layer_matches_the_oracle_of_the_original_layer(case, sparse):
    name, N, H, W, Ci, Co, K, s, p, d, f = case
    gelu = "gelu" in name
    spec = synth.LayerSpec(name, N, H, W, Ci, Co, K, K, s, p, d, relu=not gelu, gelu=gelu, w_std="fan_in", config=13,
                           index=Ci + Co + K + f)
    inp = synth.make_inputs(spec)
    res = parity.make_residual(spec, None) if "res" in name else None
    desc = api.desc_from_spec(spec)
    folded = api.ssconv_fold_desc(desc, f)
    w = inp.w.to(DEV)
    w_f, b_f = api.ssconv_fold_weights(desc, f, w, inp.bias.to(DEV))
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    y = torch.full((N, spec.H_out, spec.W_out, Co), float("nan"), dtype=torch.bfloat16, device=DEV)
    r = res.to(DEV) if res is not None else None
    mask = None
    if sparse:
        pat = api.ssconv_select_mask(api.MASK_MAGNITUDE_BF16, w, spec.G)
        pat_f, _ = api.ssconv_fold_weights(desc, f, pat)
        w_comp, meta = api.ssconv_compress(folded, w_f, pat_f)
        api.ssconv_forward(folded, inp.x.to(DEV), w_comp, meta, b_f, y=y, dev_status=status, residual=r)
        mask = masks.mask_from_pattern(parity.oracle_pattern(inp), tuple(inp.w.shape))
    else:
        api.ssconv_forward_dense(folded, inp.x.to(DEV), w_f, b_f, y=y, dev_status=status, residual=r)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    import dataclasses
    shp = dataclasses.replace(parity.oracle_shape(spec), relu=False)
    ref = conv2d_f64(shp, synth.bf16_bits(inp.x), synth.bf16_bits(inp.w), mask=mask, bias=inp.bias.numpy())
    if res is not None:
        ref = ref + parity.bf16_tensor_to_f64(res)
    ref = parity.gelu_f64(ref) if gelu else np.maximum(ref, 0.0)
    rel, mx = parity.errors(parity.bf16_tensor_to_f64(y), ref)
    assert rel <= parity.REL_FRO_TOL and mx <= parity.MAX_ABS_TOL, f"rel={rel:.3e} max={mx:.3e}"


def _s2d_numpy(x_bits, s, pad, Hb, Wb, c_pad):
    N, H, W, C = x_bits.shape
    y = np.zeros((N, Hb, Wb, c_pad), dtype=np.uint16)
    for r in range(Hb):
        for q in range(Wb):
            for bh in range(s):
                for bw in range(s):
                    h, w = s * r - pad + bh, s * q - pad + bw
                    if 0 <= h < H and 0 <= w < W:
                        y[:, r, q, (bh * s + bw) * C:(bh * s + bw + 1) * C] = x_bits[:, h, w, :]
    return y


@pytest.mark.parametrize("shape,s,pad,Hb,Wb,c_pad", [
    ((2, 16, 24, 3), 2, 3, 11, 16, 12),    # RGB, width a multiple of 8: the staged two-row kernel
    ((3, 9, 8, 3), 2, 1, 6, 6, 12),        # the same kernel, rows past the bottom edge
    ((2, 10, 11, 3), 2, 3, 8, 9, 12),      # odd width: the generic kernel at 8-byte granularity
    ((1, 7, 9, 1), 3, 2, 4, 5, 12),        # one channel, blocks of 3 x 3
    ((64, 7, 7, 3), 2, 0, 4, 4, 12),       # a weight tensor
    ((2, 32, 24, 3), 4, 0, 8, 6, 48),      # RGB, blocks of 4 x 4 (a patchify stem): the staged four-row kernel
    ((3, 18, 16, 3), 4, 3, 7, 6, 48),      # the same with padding on every side and rows past the bottom edge
    ((1, 16, 40, 3), 4, 2, 4, 7, 48),      # fewer block columns than the image has: the row's tail is dropped
    ((2, 12, 10, 3), 4, 1, 4, 4, 48),      # width not a multiple of 8: the generic kernel
])
def test_space_to_depth_of_few_channel_images_is_bit_exact(shape, s, pad, Hb, Wb, c_pad):
    g = torch.Generator().manual_seed(synth.SEED_BASE + 3500 + shape[1] + shape[2])
    x = torch.randn(shape, generator=g).to(torch.bfloat16)
    band = 64
    buf = torch.full((shape[0] * Hb * Wb * c_pad + 2 * band,), -3.0, dtype=torch.bfloat16, device=DEV)
    y = buf[band:-band].view(shape[0], Hb, Wb, c_pad)
    api.ssconv_space_to_depth(x.to(DEV), s, pad, Hb, Wb, c_pad, y=y)
    torch.cuda.synchronize()
    np.testing.assert_array_equal(synth.bf16_bits(y.cpu()), _s2d_numpy(synth.bf16_bits(x), s, pad, Hb, Wb, c_pad))
    assert bool((buf[:band] == -3.0).all()) and bool((buf[-band:] == -3.0).all())
