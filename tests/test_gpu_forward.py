"""GPU parity of the sparse and dense forward kernels against the fp64 oracle."""
import numpy as np
import pytest
import torch

from paper_2411_00288_b200 import api, synth
from tests import parity

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _assert_ok(rel, mx, what):
    assert rel <= parity.REL_FRO_TOL and mx <= parity.MAX_ABS_TOL, f"{what}: rel_fro={rel:.3e} max_abs={mx:.3e}"


def test_config1_sparse_and_dense():
    spec = synth.config_layers(1)[0]
    _assert_ok(*parity.check_layer(spec, DEV, sparse=True), "config 1 sparse")
    _assert_ok(*parity.check_layer(spec, DEV, sparse=False), "config 1 dense")


SWEEP = [
    # name                      N  H   W   Ci   Co  KH KW s  p  d
    ("pw_64",                   2, 9,  7,  64,  64, 1, 1, 1, 0, 1),
    ("pw_ragged_96to136",       3, 11, 5,  96, 136, 1, 1, 1, 0, 1),
    ("pw_s2",                   2, 10, 10, 64, 128, 1, 1, 2, 0, 1),
    ("c3_s1p1",                 2, 12, 9,  64, 128, 3, 3, 1, 1, 1),
    ("c3_s2p1",                 2, 13, 12, 128, 64, 3, 3, 2, 1, 1),
    ("c3_nopad",                1, 10, 10, 64,  64, 3, 3, 1, 0, 1),
    ("c3_dil2",                 1, 12, 12, 64,  64, 3, 3, 1, 2, 2),
    ("c5_p2",                   1, 9,  9,  32,  40, 5, 5, 1, 2, 1),
    ("c3_small_channels",       2, 8,  8,  8,   8,  3, 3, 1, 1, 1),
    ("c3_7x7_maps_wrap_images", 9, 7,  7,  128, 256, 3, 3, 1, 1, 1),
    ("pw_deepK",                1, 6,  6,  1024, 64, 1, 1, 1, 0, 1),
    # 8 input channels: the dense kernel packs 8 filter taps into a k-block (a channel-padded RGB stem)
    ("stem_7x7_s2_c8",          2, 30, 34, 8,  64,  7, 7, 2, 3, 1),
    ("pw_c8",                   2, 9,  9,  8,  16,  1, 1, 1, 0, 1),
    ("c4x4_c8_even_taps",       1, 12, 12, 8,  136, 4, 4, 1, 1, 1),
    # degenerate extents: a single pixel, a single row, a filter larger than the image
    ("one_pixel",               1, 1,  1,  8,   8,  1, 1, 1, 0, 1),
    ("one_row_wide",            1, 1,  301, 64, 64, 1, 1, 1, 0, 1),
    ("filter_exceeds_image",    2, 2,  3,  16,  24, 5, 5, 1, 2, 1),
    ("stride3_pad0",            1, 10, 13, 32,  40, 3, 3, 3, 0, 1),
]


@pytest.mark.parametrize("case", SWEEP, ids=[c[0] for c in SWEEP])
@pytest.mark.parametrize("sparse", [True, False], ids=["sparse", "dense"])
def test_shape_sweep(case, sparse):
    name, N, H, W, Ci, Co, KH, KW, s, p, d = case
    spec = synth.LayerSpec(name, N, H, W, Ci, Co, KH, KW, s, p, d, relu=(Co % 16 == 0), w_std="fan_in",
                           mask_source="magnitude", config=9, index=SWEEP.index(case))
    _assert_ok(*parity.check_layer(spec, DEV, sparse=sparse), name)


def test_no_bias_no_relu_and_gumbel_logit_masks():
    spec = synth.LayerSpec("nobias", 2, 14, 14, 128, 128, 3, 3, 1, 1, 1, relu=False, has_bias=False, w_std="he",
                           mask_source="gumbel_logits", config=9, index=50)
    _assert_ok(*parity.check_layer(spec, DEV, sparse=True), "no bias")


def test_sparse_equals_dense_on_masked_weights():
    """Eq. 6: the sparse kernel on (values, metadata) and the dense kernel on M .* W agree closely."""
    spec = synth.LayerSpec("x", 2, 14, 14, 128, 128, 3, 3, 1, 1, 1, config=9, index=51)
    inp = synth.make_inputs(spec)
    desc = api.desc_from_spec(spec)
    x, w, b = inp.x.to(DEV), inp.w.to(DEV), inp.bias.to(DEV)
    pat = api.ssconv_select_mask(api.MASK_MAGNITUDE_BF16, w, spec.G)
    w_comp, meta = api.ssconv_compress(desc, w, pat)
    w_masked, _ = api.ssconv_decompress(desc, w_comp, meta)
    ys = api.ssconv_forward(desc, x, w_comp, meta, b)
    yd = api.ssconv_forward_dense(desc, x, w_masked, b)
    torch.cuda.synchronize()
    assert (ys.float() - yd.float()).abs().max().item() <= 2 ** -6


def test_all_ones_input_closed_form_borders():
    """x == 1, w == 2^-3: y = bias + 2^-3 * (C_in/2) * #taps inside the image, exactly representable."""
    N, H, W, C, Co, K = 1, 9, 10, 64, 64, 3
    desc = api.make_desc(N, H, W, C, Co, K, K, 1, 1, 1, bias=False, relu=False)
    x = torch.ones((N, H, W, C), dtype=torch.bfloat16, device=DEV)
    w = torch.full((Co, K, K, C), 0.125, dtype=torch.bfloat16, device=DEV)
    pat = torch.randint(0, 6, (Co * K * K * C // 4,), dtype=torch.uint8, device=DEV)
    w_comp, meta = api.ssconv_compress(desc, w, pat)
    y = api.ssconv_forward(desc, x, w_comp, meta).float().cpu().numpy()
    for ho in range(H):
        for wo in range(W):
            taps = sum(1 for kh in range(K) for kw in range(K) if 0 <= ho - 1 + kh < H and 0 <= wo - 1 + kw < W)
            assert (y[0, ho, wo, :] == 0.125 * (C // 2) * taps).all()


# ---------------------------------------------------------------------------------------------
# fused residual: y = act(bias + conv + residual)
RES_CASES = [
    # name                      N  H   W   Ci   Co  KH KW s  p  d
    ("res_pw_256to64",          2, 14, 14, 256, 64,  1, 1, 1, 0, 1),
    ("res_pw_64to256",          3, 9,  11, 64,  256, 1, 1, 1, 0, 1),
    ("res_c3_ragged_136",       2, 12, 9,  64,  136, 3, 3, 1, 1, 1),
    ("res_c3_s2",               2, 13, 12, 128, 64,  3, 3, 2, 1, 1),
    ("res_small_channels",      2, 8,  8,  8,   8,   3, 3, 1, 1, 1),
]


@pytest.mark.parametrize("case", RES_CASES, ids=[c[0] for c in RES_CASES])
@pytest.mark.parametrize("sparse", [True, False], ids=["sparse", "dense"])
def test_residual_epilogue(case, sparse):
    name, N, H, W, Ci, Co, KH, KW, s, p, d = case
    spec = synth.LayerSpec(name, N, H, W, Ci, Co, KH, KW, s, p, d, relu=(Co != 136), w_std="fan_in",
                           mask_source="magnitude", config=9, index=60 + RES_CASES.index(case))
    _assert_ok(*parity.check_layer(spec, DEV, sparse=sparse, residual=True), name)


def test_residual_in_place_and_wide_tiles():
    """A layer wide enough for 240-position tiles and several pieces per group, with the residual
    read from the output buffer itself (y += conv, as a skip connection updated in place)."""
    spec = synth.LayerSpec("res_inplace", 1, 188, 188, 64, 64, 3, 3, 1, 1, 1, relu=True, w_std="fan_in",
                           mask_source="magnitude", config=9, index=70)
    inp = synth.make_inputs(spec)
    res = parity.make_residual(spec)
    desc = api.desc_from_spec(spec)
    x, w, b = inp.x.to(DEV), inp.w.to(DEV), inp.bias.to(DEV)
    pat = api.ssconv_select_mask(api.MASK_MAGNITUDE_BF16, w, spec.G)
    w_comp, meta = api.ssconv_compress(desc, w, pat)
    y_sep = api.ssconv_forward(desc, x, w_comp, meta, b, residual=res.to(DEV))
    y_inplace = res.to(DEV).clone()
    api.ssconv_forward(desc, x, w_comp, meta, b, y=y_inplace, residual=y_inplace)
    torch.cuda.synchronize()
    assert torch.equal(y_sep, y_inplace)
    assert api.ssconv_plan(desc, True)["tile_positions"] == 240
    _assert_ok(*parity.check_layer(spec, DEV, sparse=True, sample=30000, residual=True), "res_inplace")


# ---------------------------------------------------------------------------------------------
# GELU epilogue (the activation of ConvNeXt's point-wise expand layers)
GELU_CASES = [
    ("gelu_pw_96to384",   2, 14, 14, 96,  384, 1, 1, 1, 0, 1),
    ("gelu_c3_64to136",   2, 12, 9,  64,  136, 3, 3, 1, 1, 1),
]


@pytest.mark.parametrize("case", GELU_CASES, ids=[c[0] for c in GELU_CASES])
@pytest.mark.parametrize("sparse", [True, False], ids=["sparse", "dense"])
@pytest.mark.parametrize("residual", [False, True], ids=["plain", "residual"])
def test_gelu_epilogue(case, sparse, residual):
    name, N, H, W, Ci, Co, KH, KW, s, p, d = case
    spec = synth.LayerSpec(name, N, H, W, Ci, Co, KH, KW, s, p, d, gelu=True, w_std="fan_in",
                           mask_source="magnitude", config=9, index=80 + GELU_CASES.index(case))
    _assert_ok(*parity.check_layer(spec, DEV, sparse=sparse, residual=residual), name)


def test_gelu_over_every_bf16_input_up_to_8():
    """Every finite bf16 value of magnitude up to 8 goes through a 1x1 convolution with identity weights:
    the output must be GELU(x) = x Phi(x) from erf in fp64, to one bf16 rounding (2^-9 relative; 2^-8 is
    allowed) plus 2e-6 absolute for the kernel's fp32 evaluation of erf."""
    from scipy.special import erf
    bits = np.arange(0, 0x4100 + 1, dtype=np.uint16)                       # +0 .. 8.0
    bits = np.concatenate([bits, bits | 0x8000]).astype(np.uint16)         # and the negatives
    n = (bits.size + 7) // 8 * 8
    allb = np.zeros(n, dtype=np.uint16)
    allb[:bits.size] = bits
    x = torch.from_numpy(allb.view(np.int16)).view(torch.bfloat16).reshape(1, 1, n // 8, 8)
    w = torch.zeros((8, 1, 1, 8), dtype=torch.bfloat16)
    for c in range(8):
        w[c, 0, 0, c] = 1.0
    desc = api.make_desc(1, 1, n // 8, 8, 8, 1, 1, bias=False, gelu=True)
    y = api.ssconv_forward_dense(desc, x.to(DEV), w.to(DEV), None).float().cpu().numpy().reshape(-1)[:bits.size]
    xv = x.float().numpy().reshape(-1)[:bits.size].astype(np.float64)
    ref = 0.5 * xv * (1.0 + erf(xv / np.sqrt(2.0)))
    err = np.abs(y - ref)
    bad = err > 2.0 ** -8 * np.abs(ref) + 2e-6
    assert not bad.any(), (xv[bad][:5], y[bad][:5], ref[bad][:5])


def test_gelu_matches_closed_values_and_flag_rules():
    """x == 1, one kept weight w per output channel and zero bias give y = GELU(w) exactly enough to tell
    GELU from ReLU and identity; RELU and GELU together are refused."""
    import ctypes
    import math
    N, H, W, C, Co = 1, 4, 4, 8, 8
    desc = api.make_desc(N, H, W, C, Co, 1, 1, bias=False, gelu=True)
    x = torch.ones((N, H, W, C), dtype=torch.bfloat16, device=DEV)
    w = torch.zeros((Co, 1, 1, C), dtype=torch.bfloat16, device=DEV)
    vals = [-3.0, -1.0, -0.5, 0.0, 0.5, 1.0, 2.0, 4.0]
    for co, v in enumerate(vals):
        w[co, 0, 0, 0] = v
    y = api.ssconv_forward_dense(desc, x, w, None).float().cpu().numpy()
    for co, v in enumerate(vals):
        want = 0.5 * v * (1.0 + math.erf(v / math.sqrt(2.0)))
        assert abs(y[0, 0, 0, co] - want) <= 2 ** -8 * max(1.0, abs(want)), (v, y[0, 0, 0, co], want)
    both = api.make_desc(N, H, W, C, Co, 1, 1, bias=False, relu=True, gelu=True)
    ho, wo = ctypes.c_int32(), ctypes.c_int32()
    assert api.lib().ssconv_out_shape(ctypes.byref(both), ctypes.byref(ho), ctypes.byref(wo)) == 2  # bad descriptor
