"""Pins for the fp64 direct-convolution oracle (CPU only).

Each test fixes the oracle to something other than itself: an independent unfold +
matrix-product restatement (Eq. 5), closed forms, impulse responses, the textbook GEMM
special case, and the algebraic identities of Eq. 6 and Lemma 3.3.
"""
import numpy as np
import pytest

from oracle import masks
from oracle.conv import ConvShape, conv2d_f64, conv2d_f64_sample, out_shape
from tests.brute import bf16_to_f64, f32_to_bf16_bits, unfold_matmul_conv


def _rand_bits(rng, shape, scale=1.0):
    return f32_to_bf16_bits((rng.normal(size=shape) * scale).astype(np.float32))


CASES = [
    # N  H  W  C  Co KH KW  stride  pad     dil
    (1, 5, 5, 4, 3, 3, 3, (1, 1), (1, 1), (1, 1)),
    (2, 6, 7, 8, 5, 3, 3, (2, 2), (1, 1), (1, 1)),
    (1, 7, 5, 4, 2, 3, 3, (1, 1), (2, 2), (2, 2)),
    (2, 4, 6, 8, 4, 1, 1, (1, 1), (0, 0), (1, 1)),
    (1, 8, 8, 4, 4, 1, 1, (2, 2), (0, 0), (1, 1)),
    (1, 6, 6, 4, 3, 3, 3, (1, 1), (0, 0), (1, 1)),
    (1, 9, 7, 4, 2, 3, 2, (2, 1), (1, 0), (1, 2)),
]


@pytest.mark.parametrize("case", CASES)
def test_matches_unfold_matmul_bruteforce(case):
    N, H, W, C, Co, KH, KW, st, pd, dl = case
    rng = np.random.default_rng(hash(case) % (2 ** 32))
    x = _rand_bits(rng, (N, H, W, C))
    w = _rand_bits(rng, (Co, KH, KW, C), 0.3)
    pat = rng.integers(0, 6, size=Co * KH * KW * C // 4).astype(np.uint8)
    m = masks.mask_from_pattern(pat, w.shape)
    bias = rng.normal(size=Co).astype(np.float32)
    s = ConvShape(N, H, W, C, Co, KH, KW, st, pd, dl, relu=False)
    got = conv2d_f64(s, x, w, mask=m, bias=bias)
    ref = unfold_matmul_conv(bf16_to_f64(x), bf16_to_f64(w) * m, st, pd, dl) + bias.astype(np.float64)
    assert got.shape == ref.shape
    # both are fp64 sums of the same exact products in a different order
    assert np.allclose(got, ref, rtol=0, atol=1e-12)
    # ReLU is applied last
    got_relu = conv2d_f64(ConvShape(N, H, W, C, Co, KH, KW, st, pd, dl, relu=True), x, w, mask=m, bias=bias)
    assert np.array_equal(got_relu, np.maximum(got, 0.0))


def test_output_extent_full_padding_gives_input_size():
    # Sec. 3.3: with p = floor(k/2) and odd k the number of blocks equals b*d
    for k in (1, 3, 5, 7):
        s = ConvShape(1, 13, 9, 4, 4, k, k, (1, 1), (k // 2, k // 2))
        assert out_shape(s) == (13, 9)
    assert out_shape(ConvShape(1, 56, 56, 4, 4, 3, 3, (2, 2), (1, 1))) == (28, 28)
    assert out_shape(ConvShape(1, 224, 224, 4, 4, 7, 7, (2, 2), (3, 3))) == (112, 112)
    assert out_shape(ConvShape(1, 7, 7, 4, 4, 3, 3, (1, 1), (0, 0), (2, 2))) == (3, 3)


def test_masked_conv_equals_dense_conv_of_masked_weights_and_all_ones_is_dense():
    rng = np.random.default_rng(21)
    s = ConvShape(2, 6, 5, 8, 4, 3, 3, (1, 1), (1, 1))
    x = _rand_bits(rng, (2, 6, 5, 8))
    w = _rand_bits(rng, (4, 3, 3, 8), 0.2)
    pat = rng.integers(0, 6, size=4 * 9 * 2).astype(np.uint8)
    m = masks.mask_from_pattern(pat, w.shape)
    # Eq. 6: (M .* W) U(X) is the dense convolution of the masked weights
    assert np.array_equal(conv2d_f64(s, x, w, mask=m), conv2d_f64(s, x, masks.apply_mask(w, m)))
    # an all-ones mask changes nothing (the unmasked reformulation predicts identically)
    assert np.array_equal(conv2d_f64(s, x, w, mask=np.ones_like(m)), conv2d_f64(s, x, w))
    # masking really drops terms
    assert not np.array_equal(conv2d_f64(s, x, w, mask=m), conv2d_f64(s, x, w))


def test_unit_impulse_returns_unflipped_kernel():
    # x = delta at (h0, w0, c0): y[ho, wo, co] = w[co, h0 - ho + p, w0 - wo + p, c0] (index SUM in Eq. 4,
    # so no kernel flip); a flipped implementation would return the mirrored slice
    C, Co, K, p = 4, 3, 3, 1
    rng = np.random.default_rng(2)
    w = _rand_bits(rng, (Co, K, K, C))
    x = np.zeros((1, 5, 5, C), dtype=np.uint16)
    h0, w0, c0 = 2, 3, 1
    x[0, h0, w0, c0] = f32_to_bf16_bits(np.float32(1.0))
    y = conv2d_f64(ConvShape(1, 5, 5, C, Co, K, K, (1, 1), (p, p)), x, w)
    wf = bf16_to_f64(w)
    for ho in range(5):
        for wo in range(5):
            kh, kw = h0 - ho + p, w0 - wo + p
            for co in range(Co):
                exp = wf[co, kh, kw, c0] if (0 <= kh < K and 0 <= kw < K) else 0.0
                assert y[0, ho, wo, co] == exp
    assert not np.array_equal(wf[:, ::-1, ::-1, c0], wf[:, :, :, c0])  # the test can tell a flip


@pytest.mark.parametrize("stride,pad,dil", [(1, 1, 1), (2, 1, 1), (1, 2, 2), (1, 0, 1), (2, 3, 1)])
def test_closed_form_ones_input_counts_valid_taps(stride, pad, dil):
    # x == 1, w == 2^-3 everywhere, any legal mask: y = bias + 2^-3 * (C_in/2) * #taps inside the image
    H, W, C, Co, K = 9, 8, 8, 2, 3
    one = f32_to_bf16_bits(np.float32(1.0))
    x = np.full((1, H, W, C), one, dtype=np.uint16)
    w = np.full((Co, K, K, C), f32_to_bf16_bits(np.float32(0.125)), dtype=np.uint16)
    rng = np.random.default_rng(4)
    m = masks.mask_from_pattern(rng.integers(0, 6, size=Co * K * K * C // 4), w.shape)
    bias = np.array([0.5, -1.25], dtype=np.float32)
    s = ConvShape(1, H, W, C, Co, K, K, (stride, stride), (pad, pad), (dil, dil))
    y = conv2d_f64(s, x, w, mask=m, bias=bias)
    Ho, Wo = out_shape(s)
    for ho in range(Ho):
        for wo in range(Wo):
            taps = sum(1 for kh in range(K) for kw in range(K)
                       if 0 <= ho * stride - pad + kh * dil < H and 0 <= wo * stride - pad + kw * dil < W)
            for co in range(Co):
                assert y[0, ho, wo, co] == bias[co] + 0.125 * (C // 2) * taps


def test_pointwise_conv_is_a_matrix_product():
    rng = np.random.default_rng(8)
    N, H, W, C, Co = 2, 3, 4, 16, 6
    x = _rand_bits(rng, (N, H, W, C))
    w = _rand_bits(rng, (Co, 1, 1, C))
    y = conv2d_f64(ConvShape(N, H, W, C, Co, 1, 1), x, w)
    ref = bf16_to_f64(x).reshape(-1, C) @ bf16_to_f64(w).reshape(Co, C).T
    assert np.allclose(y.reshape(-1, Co), ref, rtol=0, atol=1e-13)


def test_linearity_and_additive_perturbation_identity():
    rng = np.random.default_rng(13)
    s = ConvShape(1, 5, 6, 8, 3, 3, 3, (1, 1), (1, 1))
    # values on a coarse dyadic grid so that sums of inputs stay exactly representable in bf16
    x1 = f32_to_bf16_bits(rng.integers(-8, 8, size=(1, 5, 6, 8)).astype(np.float32) / 4)
    x2 = f32_to_bf16_bits(rng.integers(-8, 8, size=(1, 5, 6, 8)).astype(np.float32) / 4)
    xs = f32_to_bf16_bits((bf16_to_f64(x1) + bf16_to_f64(x2)).astype(np.float32))
    w = f32_to_bf16_bits(rng.integers(-8, 8, size=(3, 3, 3, 8)).astype(np.float32) / 8)
    assert np.array_equal(conv2d_f64(s, xs, w), conv2d_f64(s, x1, w) + conv2d_f64(s, x2, w))
    # Lemma 3.3's construction: conv(x, W) + conv(x, (B-1) .* W) = conv(x, B .* W)
    m = masks.mask_from_pattern(rng.integers(0, 6, size=3 * 9 * 2), w.shape)
    dW = f32_to_bf16_bits(((m.astype(np.float64) - 1.0) * bf16_to_f64(w)).astype(np.float32))
    assert np.array_equal(conv2d_f64(s, x1, w) + conv2d_f64(s, x1, dW), conv2d_f64(s, x1, w, mask=m))


def test_sampled_evaluation_equals_full_tensor():
    rng = np.random.default_rng(17)
    s = ConvShape(2, 7, 6, 8, 5, 3, 3, (2, 2), (1, 1), relu=True)
    x = _rand_bits(rng, (2, 7, 6, 8))
    w = _rand_bits(rng, (5, 3, 3, 8), 0.3)
    m = masks.mask_from_pattern(rng.integers(0, 6, size=5 * 9 * 2), w.shape)
    bias = rng.normal(size=5).astype(np.float32)
    full = conv2d_f64(s, x, w, mask=m, bias=bias)
    idx = rng.permutation(full.size)[:97]
    assert np.array_equal(conv2d_f64_sample(s, x, w, idx, mask=m, bias=bias), full.reshape(-1)[idx])


def test_bias_is_widened_exactly_and_added_before_relu():
    x = np.zeros((1, 2, 2, 4), dtype=np.uint16)
    w = np.zeros((2, 1, 1, 4), dtype=np.uint16)
    bias = np.array([np.float32(0.1), np.float32(-0.1)], dtype=np.float32)
    y = conv2d_f64(ConvShape(1, 2, 2, 4, 2, 1, 1, relu=True), x, w, bias=bias)
    assert (y[..., 0] == np.float64(np.float32(0.1))).all() and (y[..., 1] == 0.0).all()
