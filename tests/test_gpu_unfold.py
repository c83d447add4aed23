"""GPU tests of the width unfold: bit-exact against a numpy gather written from its definition, and
the convolution identity it exists for (a KH x KW convolution = a KH x 1 convolution over the
unfolded taps) against the fp64 oracle of the original layer."""
import numpy as np
import pytest
import torch

from oracle.conv import conv2d_f64
from paper_2411_00288_b200 import api, synth
from tests import parity

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _unfold_numpy(x_bits, KW, s, p, d, c_pad):
    *lead, W, C = x_bits.shape
    Wo = (W + 2 * p - d * (KW - 1) - 1) // s + 1
    y = np.zeros((*lead, Wo, c_pad), dtype=np.uint16)
    for wo in range(Wo):
        for kw in range(KW):
            w = wo * s - p + kw * d
            if 0 <= w < W:
                y[..., wo, kw * C:(kw + 1) * C] = x_bits[..., w, :]
    return y


@pytest.mark.parametrize("shape,KW,s,p,d,c_pad", [
    ((2, 9, 13, 8), 7, 2, 3, 1, 64),
    ((1, 4, 10, 8), 3, 1, 1, 2, 24),
    ((3, 5, 6, 16), 3, 1, 0, 1, 64),
    ((64, 7, 7, 8), 7, 1, 0, 1, 64),   # a weight tensor [C_out, KH, KW, C]
    ((1, 1, 1, 8), 1, 1, 0, 1, 8),
])
def test_unfold_w_is_bit_exact(shape, KW, s, p, d, c_pad):
    g = torch.Generator().manual_seed(synth.SEED_BASE + 3300 + KW + shape[2])
    x = torch.randn(shape, generator=g).to(torch.bfloat16)
    y = api.ssconv_unfold_w(x.to(DEV), KW, s, p, d, C_pad=c_pad)
    torch.cuda.synchronize()
    ref = _unfold_numpy(synth.bf16_bits(x), KW, s, p, d, c_pad)
    assert tuple(y.shape) == ref.shape
    np.testing.assert_array_equal(synth.bf16_bits(y.cpu()), ref)


@pytest.mark.parametrize("case", [
    # name        N  H   W   Co KH KW s  p  d
    ("stem_7x7",  2, 30, 34, 64, 7, 7, 2, 3, 1),
    ("c3_s1",     2, 12, 11, 40, 3, 3, 1, 1, 1),
    ("c5_dil2",   1, 17, 16, 16, 5, 5, 1, 4, 2),
], ids=lambda c: c[0])
def test_convolution_over_unfolded_taps_matches_the_oracle_of_the_original_layer(case):
    name, N, H, W, Co, KH, KW, s, p, d = case
    spec = synth.LayerSpec(name, N, H, W, 8, Co, KH, KW, s, p, d, relu=True, w_std="he", config=8, index=40 + KW)
    inp = synth.make_inputs(spec)
    c_pad = 64
    x, w = inp.x.to(DEV), inp.w.to(DEV)
    xu = api.ssconv_unfold_w(x, KW, s, p, d, C_pad=c_pad)
    wu = api.ssconv_unfold_w(w, KW, C_pad=c_pad)
    desc = api.make_desc(N, H, spec.W_out, c_pad, Co, KH, 1, stride=(s, 1), pad=(p, 0), dil=(d, 1), bias=True, relu=True)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    y = api.ssconv_forward_dense(desc, xu, wu, inp.bias.to(DEV), dev_status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    ref = conv2d_f64(parity.oracle_shape(spec), synth.bf16_bits(inp.x), synth.bf16_bits(inp.w), bias=inp.bias.numpy())
    rel, mx = parity.errors(parity.bf16_tensor_to_f64(y), ref)
    assert rel <= parity.REL_FRO_TOL and mx <= parity.MAX_ABS_TOL, f"{name}: rel_fro={rel:.3e} max_abs={mx:.3e}"


@pytest.mark.parametrize("shape,c_pad", [((3, 17, 9, 3), 8), ((2, 5, 7, 5), 16), ((1, 4, 4, 8), 8), ((2, 3, 3, 12), 24)])
def test_pad_channels_is_a_zero_extension(shape, c_pad):
    """ssconv_pad_channels against a plain copy into a zero tensor, bit for bit."""
    g = torch.Generator().manual_seed(synth.SEED_BASE + 990 + c_pad + shape[-1])
    x = torch.randn(shape, generator=g, dtype=torch.float32).to(torch.bfloat16)
    want = torch.zeros((*shape[:-1], c_pad), dtype=torch.bfloat16)
    want[..., :shape[-1]] = x
    got = api.ssconv_pad_channels(x.to(DEV), c_pad)
    torch.cuda.synchronize()
    assert got.shape == want.shape
    assert torch.equal(got.cpu().view(torch.int16), want.view(torch.int16))


S2D_CASES = [  # N, H, W, C, block, pad, K
    (2, 20, 22, 3, 2, 3, 7),
    (1, 9, 11, 3, 2, 2, 5),
    (2, 12, 12, 1, 3, 1, 5),
    (1, 8, 8, 4, 2, 0, 4),
]


def _s2d_extents(H, W, block, pad, K):
    T = -(-K // block)
    ho = (H + 2 * pad - K) // block + 1
    wo = (W + 2 * pad - K) // block + 1
    return T, ho, wo, ho + T - 1, wo + T - 1


@pytest.mark.parametrize("case", S2D_CASES, ids=[f"{c[1]}x{c[2]}x{c[3]}_b{c[4]}p{c[5]}k{c[6]}" for c in S2D_CASES])
def test_space_to_depth_is_a_gather(case):
    """ssconv_space_to_depth against an index-by-index gather from the zero-padded image, bit for bit."""
    N, H, W, C, block, pad, K = case
    T, ho, wo, hb, wb = _s2d_extents(H, W, block, pad, K)
    c_pad = -(-block * block * C // 8) * 8
    g = torch.Generator().manual_seed(synth.SEED_BASE + 1200 + H * W + C)
    x = torch.randn((N, H, W, C), generator=g, dtype=torch.float32).to(torch.bfloat16)
    got = api.ssconv_space_to_depth(x.to(DEV), block, pad, hb, wb, c_pad)
    torch.cuda.synchronize()
    xb = x.view(torch.int16).numpy()
    want = np.zeros((N, hb, wb, c_pad), dtype=np.int16)
    for r in range(hb):
        for q in range(wb):
            for bh in range(block):
                for bw in range(block):
                    h, w = block * r - pad + bh, block * q - pad + bw
                    if 0 <= h < H and 0 <= w < W:
                        want[:, r, q, (bh * block + bw) * C:(bh * block + bw + 1) * C] = xb[:, h, w, :]
    assert np.array_equal(got.cpu().view(torch.int16).numpy(), want)


@pytest.mark.parametrize("case", [(2, 32, 32, 3, 64, 7, 2, 3), (2, 21, 19, 3, 72, 5, 2, 2), (1, 18, 18, 2, 64, 6, 3, 0)],
                         ids=["7x7s2p3", "5x5s2p2", "6x6s3p0"])
def test_strided_convolution_through_space_to_depth_matches_oracle(case):
    """A K x K stride-s convolution over a few channels run as space-to-depth + a T x 1 convolution on a
    sliding-window view (ssconv_forward_dense_strided), against the oracle of the original layer."""
    N, H, W, C, Co, K, s, pad = case
    spec = synth.LayerSpec("s2d_layer", N, H, W, C, Co, K, K, s, pad, 1, relu=True, w_std="fan_in", config=9,
                           index=60 + K)
    g = torch.Generator().manual_seed(spec.seed)
    x = torch.randn((N, H, W, C), generator=g, dtype=torch.float32).to(torch.bfloat16)
    w = (torch.randn((Co, K, K, C), generator=g, dtype=torch.float32) / (K * K * C) ** 0.5).to(torch.bfloat16)
    bias = torch.randn((Co,), generator=g, dtype=torch.float32) * 0.1
    T, ho, wo, hb, wb = _s2d_extents(H, W, s, pad, K)
    c_pad = -(-s * s * C // 8) * 8
    xs = api.ssconv_space_to_depth(x.to(DEV), s, pad, hb, wb, c_pad)
    ws = api.ssconv_space_to_depth(w.to(DEV), s, 0, T, T, c_pad)
    desc = api.make_desc(N, hb, wo, T * c_pad, Co, T, 1, stride=1, pad=0, bias=True, relu=True)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    y = api.ssconv_forward_dense_strided(desc, xs, (c_pad, wb * c_pad, hb * wb * c_pad), ws, bias.to(DEV), dev_status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0 and tuple(y.shape) == (N, ho, wo, Co)
    ref = conv2d_f64(parity.oracle_shape(spec), synth.bf16_bits(x), synth.bf16_bits(w), mask=None, bias=bias.numpy())
    rel, mx = parity.errors(parity.bf16_tensor_to_f64(y), ref)
    assert rel <= parity.REL_FRO_TOL and mx <= parity.MAX_ABS_TOL, f"rel={rel:.3e} max={mx:.3e}"
