"""Grouped and depthwise convolutions, layer normalisation, and a ConvNeXt-shaped block chained through
the library, against the fp64 oracle.

Sec. 4 of the paper masks the dense convolutions of ResNets and ConvNeXts and leaves grouped
(depthwise) convolutions dense; the block test chains depthwise 7x7 (dense) -> layer norm -> 1x1 expand
(2:4 masked, GELU) -> 1x1 project (2:4 masked, layer scale folded into weights and bias, residual fused),
each step checked against its oracle on the bf16 input the step before produced (teacher-forced).
"""
import numpy as np
import pytest
import torch

from oracle import blocks, masks
from oracle.conv import ConvShape, conv2d_f64
from paper_2411_00288_b200 import api, synth
from tests import parity

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _bits(t):
    return synth.bf16_bits(t.cpu())


GROUPED = [  # N, H, W, C_in, C_out, K, stride, pad, groups
    (2, 14, 14, 128, 128, 3, 1, 1, 4),     # 32 channels per group: half-filled k-blocks, 32 of 128 rows per tile
    (2, 14, 14, 256, 512, 1, 1, 0, 2),
    (2, 15, 13, 64, 144, 3, 2, 1, 2),      # ragged: 72 output channels per group
    (1, 9, 9, 64, 64, 3, 1, 1, 8),         # 8 channels per group
]


def _drawn_grouped(count=10, seed=2411_00294):
    """A seeded draw on top of the list above: 2 to 6 groups, 8 to 72 input and 8 to 136 output channels per group."""
    rng = np.random.default_rng(seed)
    out = []
    while len(out) < count:
        groups = int(rng.choice([2, 3, 4, 6]))
        ci, co = int(rng.choice([8, 16, 24, 40, 64, 72])), int(rng.choice([8, 16, 40, 64, 72, 136]))
        K = int(rng.choice([1, 3, 3, 5]))
        s = int(rng.choice([1, 1, 2]))
        p = int(rng.integers(0, K))
        N, H, W = int(rng.integers(1, 4)), int(rng.integers(5, 20)), int(rng.integers(5, 20))
        out.append((N, H, W, groups * ci, groups * co, K, s, p, groups))
    return out


GROUPED = GROUPED + _drawn_grouped()


@pytest.mark.parametrize("case", GROUPED, ids=[f"g{c[8]}_{c[3]}to{c[4]}_k{c[5]}s{c[6]}p{c[7]}_{c[1]}x{c[2]}" for c in GROUPED])
@pytest.mark.parametrize("sparse", [True, False], ids=["sparse", "dense"])
def test_grouped_convolution_matches_oracle(case, sparse):
    N, H, W, Ci, Co, K, s, p, groups = case
    g = torch.Generator().manual_seed(synth.SEED_BASE + 3000 + Ci + Co + groups)
    x = torch.randn((N, H, W, Ci), generator=g).to(torch.bfloat16)
    w = (torch.randn((Co, K, K, Ci // groups), generator=g) / (K * K * Ci // groups) ** 0.5).to(torch.bfloat16)
    bias = torch.randn((Co,), generator=g) * 0.1
    desc = api.make_desc(N, H, W, Ci, Co, K, K, s, p, bias=True, relu=True)
    shape = ConvShape(N, H, W, Ci, Co, K, K, (s, s), (p, p), (1, 1), relu=True)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    ho, wo = api.ssconv_out_shape(desc)
    # the output between sentinel bands: a group's stores must stay inside its channel slice and the tensor
    band = 4096
    buf = torch.full((N * ho * wo * Co + 2 * band,), -7.0, dtype=torch.bfloat16, device=DEV)
    y = buf[band:band + N * ho * wo * Co].view(N, ho, wo, Co)
    mask = None
    if sparse:
        G = w.numel() // 4
        pat = api.ssconv_select_mask(api.MASK_MAGNITUDE_BF16, w.to(DEV), G)
        w_comp, meta = api.ssconv_compress_grouped(desc, groups, w.to(DEV), pat)
        api.ssconv_forward_grouped(desc, groups, x.to(DEV), w_comp, meta, bias.to(DEV), y=y, dev_status=status)
        pat_ref = masks.select_from_magnitude(_bits(w))
        assert np.array_equal(pat.cpu().numpy(), pat_ref)
        mask = masks.mask_from_pattern(pat_ref, tuple(w.shape))
        # each group's part of the blobs reads back as that group's masked weights
        sub = api.make_desc(N, H, W, Ci // groups, Co // groups, K, K, s, p)
        sz = api.ssconv_sizes(sub)
        wb, _ = api.ssconv_decompress(sub, w_comp[sz.w_comp_bytes:2 * sz.w_comp_bytes].clone(), meta[sz.meta_bytes:2 * sz.meta_bytes].clone())
        want = masks.apply_mask(_bits(w), mask)[Co // groups:2 * (Co // groups)]
        assert np.array_equal(_bits(wb), want)
    else:
        api.ssconv_forward_dense_grouped(desc, groups, x.to(DEV), w.to(DEV), bias.to(DEV), y=y, dev_status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    assert bool((buf[:band] == -7.0).all()) and bool((buf[-band:] == -7.0).all()) and bool((y >= 0).all())
    ref = blocks.grouped_conv2d_f64(shape, groups, _bits(x), _bits(w), mask=mask, bias=bias.numpy())
    rel, mx = parity.errors(parity.bf16_tensor_to_f64(y), ref)
    assert rel <= parity.REL_FRO_TOL and mx <= parity.MAX_ABS_TOL, f"rel={rel:.3e} max={mx:.3e}"


@pytest.mark.parametrize("case", [(2, 14, 14, 96, 7, 1, 3, 1), (2, 15, 13, 64, 3, 2, 1, 1), (1, 12, 12, 8, 3, 1, 2, 2),
                                  (3, 7, 7, 64, 7, 1, 3, 1), (1, 19, 21, 32, 5, 1, 2, 1), (2, 9, 11, 32, 3, 1, 0, 1),
                                  (1, 10, 13, 160, 7, 1, 1, 1), (1, 17, 9, 40, 7, 1, 3, 1), (2, 33, 18, 32, 7, 1, 5, 1)],
                         ids=["7x7", "3x3s2", "3x3d2", "7x7_map7_tile_tails", "5x5_c32", "3x3_pad0", "7x7_pad1", "7x7_c40_row_runs",
                              "7x7_pad5"])
def test_depthwise_matches_oracle(case):
    # unit-stride square filters on channel counts that are multiples of 32 run on the tile kernel (4 x 8 outputs
    # per thread), other unit-stride ones on the row-run kernel, the rest on the generic one
    N, H, W, C, K, s, p, d = case
    g = torch.Generator().manual_seed(synth.SEED_BASE + 3100 + C + K)
    x = torch.randn((N, H, W, C), generator=g).to(torch.bfloat16)
    w = (torch.randn((K, K, C), generator=g) / K).to(torch.bfloat16)
    bias = torch.randn((C,), generator=g) * 0.1
    desc = api.make_desc(N, H, W, C, C, K, K, s, p, d, bias=True, relu=False)
    y = api.ssconv_depthwise(desc, x.to(DEV), w.to(DEV), bias.to(DEV))
    torch.cuda.synchronize()
    shape = ConvShape(N, H, W, C, C, K, K, (s, s), (p, p), (d, d), relu=False)
    ref = blocks.depthwise_conv2d_f64(shape, _bits(x), _bits(w), bias=bias.numpy())
    rel, mx = parity.errors(parity.bf16_tensor_to_f64(y), ref)
    assert rel <= parity.REL_FRO_TOL and mx <= parity.MAX_ABS_TOL, f"rel={rel:.3e} max={mx:.3e}"


@pytest.mark.parametrize("C", [96, 192, 40])
def test_layernorm_matches_oracle(C):
    g = torch.Generator().manual_seed(synth.SEED_BASE + 3200 + C)
    x = (torch.randn((3, 7, 5, C), generator=g) * 2 + 0.5).to(torch.bfloat16)
    gamma, beta = torch.randn((C,), generator=g) * 0.5 + 1.0, torch.randn((C,), generator=g) * 0.2
    y = api.ssconv_layernorm(x.to(DEV), gamma.to(DEV), beta.to(DEV), 1e-6)
    torch.cuda.synchronize()
    ref = blocks.layernorm_f64(parity.bf16_tensor_to_f64(x), gamma.numpy(), beta.numpy(), 1e-6)
    # fp32 statistics and one rounding to bf16 (2^-9 relative) of values up to about 4 sigma
    err = np.abs(parity.bf16_tensor_to_f64(y) - ref)
    assert (err <= 2.0 ** -8 * np.abs(ref) + 1e-3).all(), err.max()


def test_convnext_block_chains_through_the_library():
    N, H, W, C = 4, 14, 14, 96
    g = torch.Generator().manual_seed(synth.SEED_BASE + 3300)
    x = torch.randn((N, H, W, C), generator=g).to(torch.bfloat16)
    w_dw = (torch.randn((7, 7, C), generator=g) / 7).to(torch.bfloat16)
    b_dw = torch.randn((C,), generator=g) * 0.1
    gamma, beta = torch.ones(C) + 0.1 * torch.randn((C,), generator=g), 0.1 * torch.randn((C,), generator=g)
    w1 = (torch.randn((4 * C, 1, 1, C), generator=g) / C ** 0.5).to(torch.bfloat16)
    b1 = torch.randn((4 * C,), generator=g) * 0.1
    layer_scale = 0.5
    w2 = (torch.randn((C, 1, 1, 4 * C), generator=g) * layer_scale / (4 * C) ** 0.5).to(torch.bfloat16)   # layer scale folded in
    b2 = torch.randn((C,), generator=g) * 0.1 * layer_scale
    xd = x.to(DEV)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    d_dw = api.make_desc(N, H, W, C, C, 7, 7, 1, 3, bias=True, relu=False)
    d1 = api.make_desc(N, H, W, C, 4 * C, 1, 1, bias=True, gelu=True)
    d2 = api.make_desc(N, H, W, 4 * C, C, 1, 1, bias=True, relu=False)
    t0 = api.ssconv_depthwise(d_dw, xd, w_dw.to(DEV), b_dw.to(DEV))
    t1 = api.ssconv_layernorm(t0, gamma.to(DEV), beta.to(DEV), 1e-6)
    p1 = api.ssconv_select_mask(api.MASK_MAGNITUDE_BF16, w1.to(DEV), w1.numel() // 4)
    c1 = api.ssconv_compress(d1, w1.to(DEV), p1)
    t2 = api.ssconv_forward(d1, t1, c1[0], c1[1], b1.to(DEV), dev_status=status)
    p2 = api.ssconv_select_mask(api.MASK_MAGNITUDE_BF16, w2.to(DEV), w2.numel() // 4)
    c2 = api.ssconv_compress(d2, w2.to(DEV), p2)
    out = api.ssconv_forward(d2, t2, c2[0], c2[1], b2.to(DEV), dev_status=status, residual=xd)   # x + scale * mlp(...)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    # teacher-forced oracles
    s_dw = ConvShape(N, H, W, C, C, 7, 7, (1, 1), (3, 3), (1, 1), relu=False)
    r0 = blocks.depthwise_conv2d_f64(s_dw, _bits(x), _bits(w_dw), bias=b_dw.numpy())
    assert parity.errors(parity.bf16_tensor_to_f64(t0), r0)[0] <= parity.REL_FRO_TOL
    r1 = blocks.layernorm_f64(parity.bf16_tensor_to_f64(t0), gamma.numpy(), beta.numpy(), 1e-6)
    assert np.abs(parity.bf16_tensor_to_f64(t1) - r1).max() <= 2.0 ** -8 * np.abs(r1).max() + 1e-3
    m1 = masks.mask_from_pattern(masks.select_from_magnitude(_bits(w1)), tuple(w1.shape))
    s1 = ConvShape(N, H, W, C, 4 * C, 1, 1, relu=False)
    r2 = parity.gelu_f64(conv2d_f64(s1, _bits(t1), _bits(w1), mask=m1, bias=b1.numpy()))
    rel, mx = parity.errors(parity.bf16_tensor_to_f64(t2), r2)
    assert rel <= parity.REL_FRO_TOL and mx <= parity.MAX_ABS_TOL, f"expand: rel={rel:.3e} max={mx:.3e}"
    m2 = masks.mask_from_pattern(masks.select_from_magnitude(_bits(w2)), tuple(w2.shape))
    s2 = ConvShape(N, H, W, 4 * C, C, 1, 1, relu=False)
    r3 = conv2d_f64(s2, _bits(t2), _bits(w2), mask=m2, bias=b2.numpy()) + parity.bf16_tensor_to_f64(x)
    rel, mx = parity.errors(parity.bf16_tensor_to_f64(out), r3)
    assert rel <= parity.REL_FRO_TOL and mx <= parity.MAX_ABS_TOL, f"project + skip: rel={rel:.3e} max={mx:.3e}"
