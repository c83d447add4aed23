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
