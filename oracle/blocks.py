"""Oracle pieces around the masked convolution that a ConvNeXt-shaped block needs (test infrastructure
only): grouped and depthwise convolution (Sec. 4 of the paper: grouped convolutions exist in the
evaluated networks and are left dense) and layer normalisation.  fp64, written from the definitions.
"""
from __future__ import annotations

import dataclasses

import numpy as np

from .conv import ConvShape, conv2d_f64


def bf16_bits_to_f64(bits: np.ndarray) -> np.ndarray:
    return (np.asarray(bits, dtype=np.uint16).astype(np.uint32) << 16).view(np.float32).astype(np.float64)


def grouped_conv2d_f64(s: ConvShape, groups: int, x_bits, w_bits, mask=None, bias=None) -> np.ndarray:
    """A grouped convolution is, by definition, `groups` independent convolutions on channel slices:
    group g maps input channels [g C_in/groups, ...) to output channels [g C_out/groups, ...).
    w_bits: [C_out, KH, KW, C_in/groups]."""
    ci, co = s.C_in // groups, s.C_out // groups
    x = np.asarray(x_bits).reshape(s.N, s.H, s.W, s.C_in)
    w = np.asarray(w_bits).reshape(s.C_out, s.KH, s.KW, ci)
    m = None if mask is None else np.asarray(mask).reshape(w.shape)
    sub = dataclasses.replace(s, C_in=ci, C_out=co)
    outs = []
    for g in range(groups):
        outs.append(conv2d_f64(sub, np.ascontiguousarray(x[..., g * ci:(g + 1) * ci]),
                               np.ascontiguousarray(w[g * co:(g + 1) * co]),
                               mask=None if m is None else np.ascontiguousarray(m[g * co:(g + 1) * co]),
                               bias=None if bias is None else np.ascontiguousarray(bias[g * co:(g + 1) * co])))
    return np.concatenate(outs, axis=-1)


def depthwise_conv2d_f64(s: ConvShape, x_bits, w_bits, bias=None) -> np.ndarray:
    """Eq. 4 with one input channel per output channel: y[n,ho,wo,c] = sum_{kh,kw} x[n,hi,wi,c] w[kh,kw,c],
    zero outside the image.  w_bits: tap-major [KH, KW, C].  Plain loops over the taps on a padded copy."""
    assert s.C_in == s.C_out
    x = bf16_bits_to_f64(x_bits).reshape(s.N, s.H, s.W, s.C_in)
    w = bf16_bits_to_f64(w_bits).reshape(s.KH, s.KW, s.C_in)
    (sh, sw), (ph, pw), (dh, dw) = s.stride, s.pad, s.dil
    ho = (s.H + 2 * ph - dh * (s.KH - 1) - 1) // sh + 1
    wo = (s.W + 2 * pw - dw * (s.KW - 1) - 1) // sw + 1
    xp = np.zeros((s.N, s.H + 2 * ph, s.W + 2 * pw, s.C_in))
    xp[:, ph:ph + s.H, pw:pw + s.W] = x
    y = np.zeros((s.N, ho, wo, s.C_in))
    for kh in range(s.KH):
        for kw in range(s.KW):
            y += xp[:, kh * dh:kh * dh + sh * ho:sh, kw * dw:kw * dw + sw * wo:sw] * w[kh, kw]
    if bias is not None:
        y += np.asarray(bias, dtype=np.float64)
    return np.maximum(y, 0.0) if s.relu else y


def layernorm_f64(x: np.ndarray, gamma: np.ndarray, beta: np.ndarray, eps: float) -> np.ndarray:
    """Over the last axis: (x - mean) / sqrt(var + eps) * gamma + beta with the biased variance."""
    x = np.asarray(x, dtype=np.float64)
    mean = x.mean(axis=-1, keepdims=True)
    var = ((x - mean) ** 2).mean(axis=-1, keepdims=True)
    return (x - mean) / np.sqrt(var + eps) * np.asarray(gamma, dtype=np.float64) + np.asarray(beta, dtype=np.float64)
