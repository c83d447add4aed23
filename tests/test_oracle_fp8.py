"""Pins of the e4m3 part of the oracle (CPU only): the decode table against the format's landmarks and
against the library's own conversion, the quantiser against brute force over all 254 finite values,
against the library's cast, and on ties, saturation and signs; the widening to bf16."""
import numpy as np
import torch

from oracle import fp8


def test_decode_table_landmarks():
    t = fp8.e4m3_decode_table()
    assert t[0x00] == 0.0 and t[0x80] == 0.0 and np.signbit(t[0x80])
    assert t[0x38] == 1.0 and t[0xB8] == -1.0
    assert t[0x01] == 2.0 ** -9                      # smallest subnormal
    assert t[0x07] == 7 * 2.0 ** -9 and t[0x08] == 2.0 ** -6   # largest subnormal, smallest normal
    assert t[0x7E] == 448.0 and np.isnan(t[0x7F]) and np.isnan(t[0xFF])
    fin = t[:0x7F]
    assert (np.diff(fin) > 0).all()                  # codes 0..0x7E ascend strictly
    assert np.array_equal(t[0x80:0xFF], -t[0x00:0x7F])
    # every binade holds 8 equally spaced values
    for e in range(1, 15):
        v = t[8 * e:8 * e + 8]
        assert np.allclose(np.diff(v), 2.0 ** (e - 7) / 8.0, rtol=0, atol=0)


def test_decode_table_equals_the_library_conversion():
    codes = torch.arange(256, dtype=torch.int32).to(torch.uint8)
    lib = codes.view(torch.float8_e4m3fn).to(torch.float64).numpy()
    t = fp8.e4m3_decode_table()
    assert np.array_equal(np.isnan(lib), np.isnan(t))
    ok = ~np.isnan(t)
    assert np.array_equal(lib[ok], t[ok]) and np.array_equal(np.signbit(lib[ok]), np.signbit(t[ok]))


def test_quantiser_fixed_points_ties_saturation_and_signs():
    t = fp8.e4m3_decode_table()
    finite = np.array([c for c in range(256) if not np.isnan(t[c])], dtype=np.uint8)
    assert np.array_equal(fp8.quantize_e4m3(t[finite]), finite)          # every value is its own nearest
    pos = t[:0x7F]
    mid = (pos[:-1] + pos[1:]) / 2                                         # exact midpoints: ties
    q = fp8.quantize_e4m3(mid)
    assert ((q & 1) == 0).all()                                            # ... go to the even mantissa
    assert np.array_equal(q, np.where(np.arange(0x7E) % 2 == 0, np.arange(0x7E), np.arange(1, 0x7F)).astype(np.uint8))
    eps = np.nextafter(mid, np.inf) - mid
    assert np.array_equal(fp8.quantize_e4m3(mid + eps), np.arange(1, 0x7F).astype(np.uint8))
    assert np.array_equal(fp8.quantize_e4m3(mid - eps), np.arange(0, 0x7E).astype(np.uint8))
    assert np.array_equal(fp8.quantize_e4m3(np.array([449.0, 1e9, -464.0, -1e30])), np.array([0x7E, 0x7E, 0xFE, 0xFE], dtype=np.uint8))
    assert np.array_equal(fp8.quantize_e4m3(np.array([-0.0, -1e-9, 1e-9])), np.array([0x80, 0x80, 0x00], dtype=np.uint8))


def test_quantiser_is_the_nearest_value_by_brute_force_and_matches_the_library_cast():
    rng = np.random.default_rng(7)
    x = np.concatenate([rng.normal(size=20000), rng.normal(size=20000) * 40, rng.uniform(-500, 500, size=20000),
                        rng.normal(size=5000) * 1e-2]).astype(np.float32).astype(np.float64)
    q = fp8.quantize_e4m3(x)
    t = fp8.e4m3_decode_table()
    vals = t[:0x7F]
    # brute force: no finite value is strictly closer to min(|x|, 448) than the chosen one
    mag = np.minimum(np.abs(x), 448.0)
    chosen = np.abs(t[q])
    best = np.abs(vals[None, :] - mag[:, None]).min(axis=1)
    assert np.array_equal(np.abs(chosen - mag), best)
    assert np.array_equal(np.signbit(t[q]), np.signbit(x))
    # the library's cast rounds to nearest even too; it turns magnitudes beyond the format's range into NaN
    # instead of saturating, so compare inside the range
    inside = np.abs(x) <= 448.0
    lib = torch.from_numpy(x[inside].astype(np.float32)).to(torch.float8_e4m3fn).view(torch.uint8).numpy()
    assert np.array_equal(lib, q[inside])


def test_every_e4m3_value_is_a_bf16_value():
    codes = np.array([c for c in range(256) if (c & 0x7F) != 0x7F], dtype=np.uint8)
    bits = fp8.e4m3_to_bf16_bits(codes)
    back = (bits.astype(np.uint32) << 16).view(np.float32).astype(np.float64)
    assert np.array_equal(back, fp8.e4m3_decode(codes))
    assert np.array_equal(np.signbit(back), np.signbit(fp8.e4m3_decode(codes)))
