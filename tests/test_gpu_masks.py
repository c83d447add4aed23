"""GPU parity (bit-exact) of mask selection, compression and decompression against the oracle."""
import numpy as np
import pytest
import torch

from oracle import masks
from paper_2411_00288_b200 import api, synth
from tests.brute import f32_to_bf16_bits

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _bits_to_bf16_tensor(bits: np.ndarray) -> torch.Tensor:
    return torch.from_numpy(bits.astype(np.uint16).view(np.int16)).view(torch.bfloat16)


def test_select_logits_bit_exact_including_ties():
    rng = np.random.default_rng(1)
    G = 100_003  # ragged: not a multiple of the block size
    s = rng.normal(size=(G, 6)).astype(np.float32)
    s[::7, 3] = s[::7, 1]            # planted ties
    s[::11] = np.float32(0.25)       # all-equal groups
    got = api.ssconv_select_mask(api.MASK_LOGITS_F32, torch.from_numpy(s).to(DEV), G).cpu().numpy()
    assert np.array_equal(got, masks.select_from_logits(s))


def test_select_magnitude_bit_exact_including_ties_and_signed_zeros():
    rng = np.random.default_rng(2)
    G = 65_537
    w = f32_to_bf16_bits(rng.normal(size=(G, 4)).astype(np.float32))
    w[::5, 2] = w[::5, 0] ^ np.uint16(0x8000)   # equal magnitude, opposite sign
    w[::13] = 0
    w[1::13, 1] = 0x8000                         # -0
    got = api.ssconv_select_mask(api.MASK_MAGNITUDE_BF16, _bits_to_bf16_tensor(w).to(DEV), G).cpu().numpy()
    assert np.array_equal(got, masks.select_from_magnitude(w))


def test_select_empty_input_is_a_noop():
    out = api.ssconv_select_mask(api.MASK_LOGITS_F32, torch.empty((0, 6), device=DEV), 0)
    assert out.numel() == 0


def _drawn_weight_shapes(count=12, seed=2411_00293):
    """A seeded draw of weight shapes nobody picked by hand: non-square filters, channel counts with tails of 8
    to 56 in the last 64-channel chunk, output channels on both sides of one tile of 128."""
    rng = np.random.default_rng(seed)
    return [(int(rng.choice([8, 24, 72, 128, 136, 200, 264])), int(rng.integers(1, 6)), int(rng.integers(1, 6)),
             int(rng.choice([8, 16, 40, 64, 72, 104, 120, 192, 200, 328]))) for _ in range(count)]


@pytest.mark.parametrize("shape", [
    (64, 3, 3, 64),     # config-1 layer: padded rows (64 -> 128) and an odd number of k-blocks
    (136, 1, 1, 96),    # ragged C_out, C_in not a multiple of 64
    (256, 3, 3, 128),
    (8, 2, 3, 8),       # smallest legal channel counts
] + _drawn_weight_shapes())
def test_compress_roundtrip_bit_exact(shape):
    Co, KH, KW, Ci = shape
    rng = np.random.default_rng(Co * 1000 + Ci)
    w = f32_to_bf16_bits(rng.normal(size=shape).astype(np.float32))
    w[0, 0, 0, :4] = 0
    pat = rng.integers(0, 6, size=Co * KH * KW * Ci // 4).astype(np.uint8)
    desc = api.make_desc(1, 8, 8, Ci, Co, KH, KW, 1, 0)
    w_comp, meta = api.ssconv_compress(desc, _bits_to_bf16_tensor(w).to(DEV), torch.from_numpy(pat).to(DEV))
    w_back, pat_back = api.ssconv_decompress(desc, w_comp, meta)
    torch.cuda.synchronize()
    expect = masks.apply_mask(w, masks.mask_from_pattern(pat, shape))
    got = w_back.cpu().view(torch.int16).numpy().view(np.uint16)
    assert np.array_equal(got, expect)
    assert np.array_equal(pat_back.cpu().numpy(), pat)
    # the value blob holds exactly the oracle's kept pairs (logical form of Fig. 1), zeros in the padding
    vals, codes = masks.logical_compress(w, pat)
    blob = w_comp.cpu().numpy().view(np.uint16)
    cblocks = (Ci + 63) // 64
    kb = KH * KW * cblocks
    kbp = (kb + 1) // 2 * 2
    Mp = (Co + 127) // 128 * 128
    blob = blob.reshape(Mp, kbp, 32)
    vals = vals.reshape(Co, KH * KW, Ci // 4, 2)
    total_kept = 0
    for b in range(kb):
        cc, tap = divmod(b, KH * KW)  # k-blocks are numbered chunk-major
        ng = min(16, Ci // 4 - 16 * cc)
        assert np.array_equal(blob[:Co, b, :2 * ng], vals[:, tap, 16 * cc:16 * cc + ng, :].reshape(Co, -1))
        total_kept += blob[:Co, b, :2 * ng].size
        assert (blob[:Co, b, 2 * ng:] == 0).all()
    assert total_kept == w.size // 2
    assert (blob[Co:] == 0).all() and (blob[:, kb:] == 0).all()
    # every metadata nibble is one of the six ascending position pairs
    m = meta.cpu().numpy()
    nib = np.concatenate([m & 0xF, m >> 4])
    assert set(np.unique(nib)) <= {0x4, 0x8, 0xC, 0x9, 0xD, 0xE}


def test_compress_treats_out_of_range_patterns_as_pattern_zero():
    """The pattern array lives on the device and cannot be checked on the host: values outside 0..5
    must still give well-formed blobs (legal metadata, the kept values of pattern 0)."""
    shape = (64, 1, 1, 64)
    rng = np.random.default_rng(5)
    w = f32_to_bf16_bits(rng.normal(size=shape).astype(np.float32))
    G = 64 * 64 // 4
    pat = rng.integers(0, 6, size=G).astype(np.uint8)
    bad = pat.copy()
    where = rng.choice(G, size=40, replace=False)
    bad[where] = rng.choice(np.array([6, 7, 8, 31, 200, 255], dtype=np.uint8), size=40)
    fixed = pat.copy()
    fixed[where] = 0
    desc = api.make_desc(1, 8, 8, 64, 64, 1, 1, 1, 0)
    w_comp, meta = api.ssconv_compress(desc, _bits_to_bf16_tensor(w).to(DEV), torch.from_numpy(bad).to(DEV))
    w_back, pat_back = api.ssconv_decompress(desc, w_comp, meta)
    torch.cuda.synchronize()
    m = meta.cpu().numpy()
    assert set(np.unique(np.concatenate([m & 0xF, m >> 4]))) <= {0x4, 0x8, 0xC, 0x9, 0xD, 0xE}
    assert np.array_equal(pat_back.cpu().numpy(), fixed)
    expect = masks.apply_mask(w, masks.mask_from_pattern(fixed, shape))
    assert np.array_equal(w_back.cpu().view(torch.int16).numpy().view(np.uint16), expect)
