"""Pins of the grouped / depthwise convolution and layer-norm oracles (CPU only)."""
import numpy as np
import torch

from oracle import blocks
from oracle.conv import ConvShape, conv2d_f64
from tests.brute import f32_to_bf16_bits


def _rand_bits(rng, shape, std=1.0):
    return f32_to_bf16_bits((rng.normal(size=shape) * std).astype(np.float32))


def test_grouped_with_one_group_is_the_plain_convolution_and_groups_are_block_diagonal_weights():
    rng = np.random.default_rng(1)
    s = ConvShape(2, 7, 6, 24, 16, 3, 3, (1, 1), (1, 1), (1, 1), relu=False)
    x = _rand_bits(rng, (2, 7, 6, 24))
    bias = rng.normal(size=16).astype(np.float32)
    w1 = _rand_bits(rng, (16, 3, 3, 24), 0.1)
    assert np.array_equal(blocks.grouped_conv2d_f64(s, 1, x, w1, bias=bias), conv2d_f64(s, x, w1, bias=bias))
    # textbook identity: a grouped convolution is a dense one whose weights are zero outside the diagonal blocks
    groups = 4
    wg = _rand_bits(rng, (16, 3, 3, 6), 0.1)
    dense = np.zeros((16, 3, 3, 24), dtype=np.uint16)
    for g in range(groups):
        dense[4 * g:4 * g + 4, :, :, 6 * g:6 * g + 6] = wg[4 * g:4 * g + 4]
    a = blocks.grouped_conv2d_f64(s, groups, x, wg, bias=bias)
    b = conv2d_f64(s, x, dense, bias=bias)
    assert np.allclose(a, b, rtol=0, atol=1e-12)


def test_depthwise_is_the_grouped_convolution_with_one_channel_per_group_and_no_flip():
    rng = np.random.default_rng(2)
    for (k, st, p, d) in ((7, 1, 3, 1), (3, 2, 1, 1), (3, 1, 2, 2)):
        s = ConvShape(2, 9, 8, 8, 8, k, k, (st, st), (p, p), (d, d), relu=False)
        x = _rand_bits(rng, (2, 9, 8, 8))
        w = _rand_bits(rng, (k, k, 8), 0.2)
        bias = rng.normal(size=8).astype(np.float32)
        got = blocks.depthwise_conv2d_f64(s, x, w, bias=bias)
        w_grouped = np.ascontiguousarray(np.transpose(w, (2, 0, 1)))[..., None]   # [C, KH, KW, 1]
        want = blocks.grouped_conv2d_f64(s, 8, x, w_grouped, bias=bias)
        assert np.allclose(got, want, rtol=0, atol=1e-12)
    # impulse: the output is the un-flipped filter around the impulse (cross-correlation)
    s = ConvShape(1, 5, 5, 8, 8, 3, 3, (1, 1), (1, 1), (1, 1), relu=False)
    x = np.zeros((1, 5, 5, 8), dtype=np.uint16)
    x[0, 2, 2, :] = 0x3F80
    w = _rand_bits(rng, (3, 3, 8))
    y = blocks.depthwise_conv2d_f64(s, x, w)
    wf = blocks.bf16_bits_to_f64(w)
    assert np.array_equal(y[0, 1:4, 1:4], wf[::-1, ::-1])   # y[2+a, 2+b] = w[1-a, 1-b]


def test_layernorm_moments_invariances_and_the_library_routine():
    rng = np.random.default_rng(3)
    x = rng.normal(size=(50, 96)) * 3 + 1.5
    ones, zeros = np.ones(96), np.zeros(96)
    y = blocks.layernorm_f64(x, ones, zeros, 0.0)
    assert np.allclose(y.mean(axis=-1), 0, atol=1e-12) and np.allclose((y ** 2).mean(axis=-1), 1, atol=1e-12)
    assert np.allclose(blocks.layernorm_f64(x + 7.0, ones, zeros, 0.0), y, atol=1e-10)       # shift invariance
    assert np.allclose(blocks.layernorm_f64(x * 4.0, ones, zeros, 0.0), y, atol=1e-10)       # scale invariance at eps = 0
    gamma, beta = rng.normal(size=96), rng.normal(size=96)
    want = torch.nn.functional.layer_norm(torch.from_numpy(x), (96,), torch.from_numpy(gamma), torch.from_numpy(beta), 1e-6)
    assert np.allclose(blocks.layernorm_f64(x, gamma, beta, 1e-6), want.numpy(), rtol=0, atol=1e-12)
