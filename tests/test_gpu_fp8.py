"""GPU parity of the 8-bit (e4m3) path against the oracle.

Quantisation, mask selection by magnitude and the compression round trip are bit-exact; the masked
convolution (sparse tcgen05.mma kind::f8f6f4) and its dense counterpart meet the same gates as the
bf16 path against the fp64 oracle: the e4m3 codes are widened exactly to bf16 and go through the same
direct convolution (oracle/conv_oracle.c), then the output scale is applied in fp64.  Products of e4m3
values are exact in fp32 and the accumulation is fp32 as for bf16, so the expected error is again the
one rounding of the bf16 output.
"""
import numpy as np
import pytest
import torch

from oracle import fp8, masks
from oracle.conv import ConvShape, conv2d_f64
from paper_2411_00288_b200 import api, synth
from tests import parity

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _f32_to_bf16_tensor(a):
    return torch.from_numpy(a.astype(np.float32)).to(torch.bfloat16)


def test_quantise_bit_exact_against_the_oracle():
    rng = np.random.default_rng(21)
    x = np.concatenate([rng.normal(size=50000), rng.normal(size=50000) * 60, rng.uniform(-600, 600, size=20000),
                        rng.normal(size=8000) * 1e-2, np.array([0.0, -0.0, 448.0, -448.0, 464.0, 2.0 ** -10, 1.0, -1.0])])
    x = x[: x.size // 2 * 2]
    xt = _f32_to_bf16_tensor(x)
    for scale in (1.0, 0.37, 3.0):
        got = api.ssconv_quantize_e4m3(xt.to(DEV), scale).cpu().numpy()
        prod = (xt.float().numpy() * np.float32(scale)).astype(np.float32)    # the product in fp32, as the kernel forms it
        want = fp8.quantize_e4m3(prod.astype(np.float64))
        assert np.array_equal(got, want), f"scale {scale}: {np.flatnonzero(got != want)[:5]}"


def _random_e4m3(rng, shape, std):
    return fp8.quantize_e4m3(rng.normal(size=shape) * std)


def test_select_magnitude_e4m3_bit_exact_with_ties_and_zero_signs():
    rng = np.random.default_rng(22)
    w = _random_e4m3(rng, (4096, 4), 1.0)
    w[:64] = np.array([0x38, 0xB8, 0x38, 0x38], dtype=np.uint8)   # equal magnitudes, mixed signs
    w[64:96] = np.array([0x00, 0x80, 0x00, 0x80], dtype=np.uint8)  # +0 / -0
    w[96:128, 1] = w[96:128, 3]                                   # planted ties
    got = api.ssconv_select_mask(api.MASK_MAGNITUDE_E4M3, torch.from_numpy(w).to(DEV), w.shape[0]).cpu().numpy()
    want = masks.select_from_magnitude(None, magnitudes=fp8.abs_code(w))
    assert np.array_equal(got, want)


@pytest.mark.parametrize("shape", [(64, 3, 3, 64), (136, 1, 1, 96), (256, 3, 3, 256), (8, 2, 3, 16), (128, 1, 1, 144)])
def test_compress_fp8_roundtrip_bit_exact(shape):
    Co, KH, KW, Ci = shape
    rng = np.random.default_rng(Co * 7 + Ci)
    w = _random_e4m3(rng, shape, 0.5)
    pat = rng.integers(0, 6, size=Co * KH * KW * Ci // 4).astype(np.uint8)
    desc = api.make_desc(1, 8, 8, Ci, Co, KH, KW, 1, 0)
    w_comp, meta = api.ssconv_compress_fp8(desc, torch.from_numpy(w).to(DEV), torch.from_numpy(pat).to(DEV))
    w_back, pat_back = api.ssconv_decompress_fp8(desc, w_comp, meta)
    torch.cuda.synchronize()
    m = masks.mask_from_pattern(pat, shape)
    assert np.array_equal(w_back.cpu().numpy(), np.where(m == 1, w, 0).astype(np.uint8))
    assert np.array_equal(pat_back.cpu().numpy(), pat)
    G, nv, nm = api.ssconv_sizes_fp8(desc)
    assert G == pat.size
    # the kept values: half of the dense bytes (padded to whole tiles); every metadata nibble legal
    kb = KH * KW * (-(-Ci // 128))
    assert nv == (-(-Co // 128) * 128) * ((kb + 1) // 2 * 2) * 64
    mm = meta.cpu().numpy()
    assert set(np.unique(np.concatenate([mm & 0xF, mm >> 4]))) <= {0x4, 0x8, 0xC, 0x9, 0xD, 0xE}
    blob = w_comp.cpu().numpy().reshape(-(-Co // 128) * 128, -1)
    assert (blob[Co:] == 0).all()


FP8_LAYERS = [  # name, N, H, W, C_in, C_out, K, stride, pad, dil
    ("f8_1x1_256", 3, 14, 14, 256, 256, 1, 1, 0, 1),
    ("f8_3x3_128", 2, 14, 14, 128, 128, 3, 1, 1, 1),
    ("f8_3x3_s2_64to136", 2, 15, 17, 64, 136, 3, 2, 1, 1),       # half-filled k-blocks, ragged channels
    ("f8_3x3_d2_c144", 2, 12, 12, 144, 64, 3, 1, 2, 2),          # channel tail: 128 + 16
    ("f8_1x1_c16", 2, 9, 9, 16, 64, 1, 1, 0, 1),                 # one MMA of a k-block
    ("f8_1x1_c80", 2, 9, 9, 80, 64, 1, 1, 0, 1),                 # tail needs the second MMA
    ("f8_1x1_c384_odd_kblocks", 2, 12, 12, 384, 200, 1, 1, 0, 1),
    ("f8_5x5_tiles", 1, 40, 44, 64, 64, 5, 1, 2, 1),             # several tiles per block
]


def _fp8_case(case):
    name, N, H, W, Ci, Co, K, s, p, d = case
    rng = np.random.default_rng(sum(map(ord, name)))
    fan_in = K * K * Ci
    # scales of a per-tensor quantisation: activations ~ N(0,1) mapped to +-~3.5 sigma = 448 / 128,
    # weights ~ N(0, 1/sqrt(fan_in)) likewise
    s_x, s_w = 32.0, 32.0 * np.sqrt(fan_in)
    x = fp8.quantize_e4m3(rng.normal(size=(N, H, W, Ci)) * s_x)
    w = fp8.quantize_e4m3(rng.normal(size=(Co, K, K, Ci)) / np.sqrt(fan_in) * s_w)
    bias = (rng.normal(size=Co) * 0.1).astype(np.float32)
    desc = api.make_desc(N, H, W, Ci, Co, K, K, s, p, d, bias=True, relu=True)
    shape = ConvShape(N, H, W, Ci, Co, K, K, (s, s), (p, p), (d, d), relu=False)
    return desc, shape, x, w, bias, 1.0 / (s_x * s_w)


@pytest.mark.parametrize("case", FP8_LAYERS, ids=[c[0] for c in FP8_LAYERS])
@pytest.mark.parametrize("sparse", [True, False], ids=["sparse", "dense"])
def test_forward_fp8_matches_oracle(case, sparse):
    desc, shape, x, w, bias, out_scale = _fp8_case(case)
    xd, wd, bd = torch.from_numpy(x).to(DEV), torch.from_numpy(w).to(DEV), torch.from_numpy(bias).to(DEV)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    mask = None
    if sparse:
        G = w.size // 4
        pat = api.ssconv_select_mask(api.MASK_MAGNITUDE_E4M3, wd, G)
        pat_ref = masks.select_from_magnitude(None, magnitudes=fp8.abs_code(w))
        assert np.array_equal(pat.cpu().numpy(), pat_ref)
        mask = masks.mask_from_pattern(pat_ref, w.shape)
        w_comp, meta = api.ssconv_compress_fp8(desc, wd, pat)
        y = api.ssconv_forward_fp8(desc, xd, w_comp, meta, bd, out_scale, dev_status=status)
    else:
        y = api.ssconv_forward_dense_fp8(desc, xd, wd, bd, out_scale, dev_status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    acc = conv2d_f64(shape, fp8.e4m3_to_bf16_bits(x), fp8.e4m3_to_bf16_bits(w), mask=mask, bias=None)
    ref = np.maximum(acc * np.float64(np.float32(out_scale)) + bias.astype(np.float64), 0.0)
    rel, mx = parity.errors(parity.bf16_tensor_to_f64(y), ref)
    assert np.abs(ref).max() > 0.5
    assert rel <= parity.REL_FRO_TOL and mx <= parity.MAX_ABS_TOL, f"{case[0]} sparse={sparse}: rel={rel:.3e} max={mx:.3e}"


FP8_PAIR_LAYERS = [  # run with the pair kernel forced (tiles of 256 channels on two thread blocks)
    ("f8p_3x3_256", 2, 14, 14, 256, 256, 3, 1, 1, 1),
    ("f8p_1x1_384to320", 3, 12, 12, 384, 320, 1, 1, 0, 1),       # three channel tiles: the last pair's second block idles
    ("f8p_3x3_s2_c192to264", 2, 15, 17, 192, 264, 3, 2, 1, 1),   # channel tail 128 + 64, ragged channels, stride 2
    ("f8p_1x1_c144_odd", 2, 20, 20, 144, 512, 1, 1, 0, 1),       # an odd number of k-blocks (2), tail of 16 channels
    ("f8p_3x3_tiles", 4, 28, 28, 128, 256, 3, 1, 1, 1),          # several tiles per pair
]


@pytest.mark.parametrize("case", FP8_PAIR_LAYERS, ids=[c[0] for c in FP8_PAIR_LAYERS])
@pytest.mark.parametrize("tiles_per_item", [1, 2])
def test_forward_fp8_on_thread_block_pairs_matches_oracle(case, tiles_per_item):
    desc, shape, x, w, bias, out_scale = _fp8_case(case)
    xd, wd, bd = torch.from_numpy(x).to(DEV), torch.from_numpy(w).to(DEV), torch.from_numpy(bias).to(DEV)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    pat = api.ssconv_select_mask(api.MASK_MAGNITUDE_E4M3, wd, w.size // 4)
    pat_ref = masks.select_from_magnitude(None, magnitudes=fp8.abs_code(w))
    mask = masks.mask_from_pattern(pat_ref, w.shape)
    w_comp, meta = api.ssconv_compress_fp8(desc, wd, pat)
    band = 4096
    ho, wo = api.ssconv_out_shape(desc)
    n_out = desc.N * ho * wo * desc.C_out
    buf = torch.full((n_out + 2 * band,), -7.0, dtype=torch.bfloat16, device=DEV)
    y = buf[band:band + n_out].view(desc.N, ho, wo, desc.C_out)
    api.ssconv_tune(api.TUNE_PAIR, 1)
    api.ssconv_tune(api.TUNE_PAIR_TILES, tiles_per_item - 1)        # 2: two position tiles share a group's weights
    if tiles_per_item == 2:
        api.ssconv_tune(api.TUNE_TILE_POSITIONS, 112)
    try:
        api.ssconv_forward_fp8(desc, xd, w_comp, meta, bd, out_scale, y=y, dev_status=status)
        torch.cuda.synchronize()
    finally:
        api.ssconv_tune(api.TUNE_PAIR, -1)
        api.ssconv_tune(api.TUNE_PAIR_TILES, -1)
        api.ssconv_tune(api.TUNE_TILE_POSITIONS, 0)
    assert int(status.item()) == 0
    assert bool((buf[:band] == -7.0).all()) and bool((buf[-band:] == -7.0).all()) and bool((y >= 0).all())
    acc = conv2d_f64(shape, fp8.e4m3_to_bf16_bits(x), fp8.e4m3_to_bf16_bits(w), mask=mask, bias=None)
    ref = np.maximum(acc * np.float64(np.float32(out_scale)) + bias.astype(np.float64), 0.0)
    rel, mx = parity.errors(parity.bf16_tensor_to_f64(y), ref)
    assert rel <= parity.REL_FRO_TOL and mx <= parity.MAX_ABS_TOL, f"{case[0]}: rel={rel:.3e} max={mx:.3e}"


def test_forward_fp8_argument_rules():
    desc, shape, x, w, bias, out_scale = _fp8_case(FP8_LAYERS[0])
    xd, wd = torch.from_numpy(x).to(DEV), torch.from_numpy(w).to(DEV)
    with pytest.raises(api.SsconvError):
        api.ssconv_forward_dense_fp8(desc, xd, wd, None, out_scale)                 # bias flag without bias
    nob = api.make_desc(desc.N, desc.H, desc.W, desc.C_in, desc.C_out, 1, 1, bias=False)
    with pytest.raises(api.SsconvError):
        api.ssconv_forward_dense_fp8(nob, xd, wd, None, 0.0)                        # scale must be positive
    odd = api.make_desc(1, 4, 4, 24, 64, 1, 1, bias=False)                          # C_in % 16 != 0
    with pytest.raises(api.SsconvError) as e:
        api.ssconv_sizes_fp8(odd)
    assert e.value.status == 3


def _draw_fp8_cases(count=20, seed=2411_00291):
    rng = np.random.default_rng(seed)
    cases = []
    while len(cases) < count:
        K = int(rng.choice([1, 1, 2, 3, 3, 5]))
        d = int(rng.choice([1, 1, 2]))
        s = int(rng.choice([1, 1, 2, 3]))
        p = int(rng.integers(0, d * (K - 1) + 1))
        N, H, W = int(rng.integers(1, 4)), int(rng.integers(1, 33)), int(rng.integers(1, 33))
        Ci = int(rng.choice([16, 32, 48, 64, 80, 128, 144, 192, 256, 320]))
        Co = int(rng.choice([8, 24, 64, 72, 128, 136, 200, 256, 264]))
        if H + 2 * p < d * (K - 1) + 1 or W + 2 * p < d * (K - 1) + 1:
            continue
        Ho, Wo = (H + 2 * p - d * (K - 1) - 1) // s + 1, (W + 2 * p - d * (K - 1) - 1) // s + 1
        if N * Ho * Wo * Co * K * K * Ci > 3e8:
            continue
        cases.append((f"f8r{len(cases)}_{N}x{H}x{W}x{Ci}to{Co}_k{K}s{s}p{p}d{d}", N, H, W, Ci, Co, K, s, p, d))
    return cases


FP8_RANDOM = _draw_fp8_cases()


@pytest.mark.parametrize("case", FP8_RANDOM, ids=[c[0] for c in FP8_RANDOM])
@pytest.mark.parametrize("sparse", [True, False], ids=["sparse", "dense"])
def test_forward_fp8_on_drawn_shapes_matches_oracle(case, sparse):
    """The same check on a seeded draw of shapes (channel tails of 16 to 112, ragged output channels, strides,
    dilations, paddings) nobody picked by hand."""
    desc, shape, x, w, bias, out_scale = _fp8_case(case)
    xd, wd, bd = torch.from_numpy(x).to(DEV), torch.from_numpy(w).to(DEV), torch.from_numpy(bias).to(DEV)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    mask = None
    if sparse:
        pat = api.ssconv_select_mask(api.MASK_MAGNITUDE_E4M3, wd, w.size // 4)
        pat_ref = masks.select_from_magnitude(None, magnitudes=fp8.abs_code(w))
        assert np.array_equal(pat.cpu().numpy(), pat_ref)
        mask = masks.mask_from_pattern(pat_ref, w.shape)
        w_comp, meta = api.ssconv_compress_fp8(desc, wd, pat)
        y = api.ssconv_forward_fp8(desc, xd, w_comp, meta, bd, out_scale, dev_status=status)
    else:
        y = api.ssconv_forward_dense_fp8(desc, xd, wd, bd, out_scale, dev_status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    acc = conv2d_f64(shape, fp8.e4m3_to_bf16_bits(x), fp8.e4m3_to_bf16_bits(w), mask=mask, bias=None)
    ref = np.maximum(acc * np.float64(np.float32(out_scale)) + bias.astype(np.float64), 0.0)
    rel, mx = parity.errors(parity.bf16_tensor_to_f64(y), ref)
    assert rel <= parity.REL_FRO_TOL and mx <= parity.MAX_ABS_TOL, f"{case[0]} sparse={sparse}: rel={rel:.3e} max={mx:.3e}"
