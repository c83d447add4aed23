"""CPU oracle for the mask-learning step: soft masks, their gradient, and the weight gradient
of the convolution.

TEST INFRASTRUCTURE, not a product path: only the tests, the smoke check and the
benchmark's CPU-baseline leg may import this module.  It shares no code with the CUDA
library and imports nothing from the package.  Everything is fp64 numpy.

What it restates (Sec. 3.1 and Sec. 3.3 of the paper):

* Eq. 3: the relaxed choice vector of a group, z_i = exp((g_i + log pi_i) / tau) /
  sum_k exp((g_k + log pi_k) / tau), with the Gumbel noise g drawn by the caller and passed
  in, and the trainable choice weights passed as logits l_i = log pi_i (any additive constant
  per group cancels).
* Eq. 2 with that z in place of the one-hot vector: the block b = D z of four soft mask
  entries, each in [0, 1], summing to 2.
* Eq. 6 with the soft mask: effective weights W_eff = M .* W, which the dense convolution
  (Eq. 5) then uses.  Only the choice weights are trained (Sec. 4.1); the pretrained weights
  stay as they are.
* The gradients follow from the chain rule; the paper prints none of them.  With
  G = dL/dW_eff:   dL/db_j = G_j W_j,   dL/dz_i = sum_j D[j, i] dL/db_j,
  dL/dl_i = z_i (dL/dz_i - sum_k z_k dL/dz_k) / tau   (the softmax Jacobian).
* The weight gradient of the convolution of Eq. 4: dL/dW_eff[co, kh, kw, ci] =
  sum over images and output pixels of dL/dy[n, ho, wo, co] x[n, ho s - p + kh d,
  wo s - p + kw d, ci], pixels outside the image contributing nothing (they are the zero
  padding).
* The gradient with respect to the layer's input is the adjoint of the same linear map in x.
* The choice weights are updated with AdamW (Appendix, training details: learning rate 1.0,
  momentum 0.9, weight decay 1e-4).  The update is the published one (decoupled weight decay):
  m <- b1 m + (1 - b1) g,  v <- b2 v + (1 - b2) g^2,  theta <- theta - lr (mhat / (sqrt(vhat) + eps)
  + wd theta) with the bias-corrected mhat = m / (1 - b1^t), vhat = v / (1 - b2^t).
"""
from __future__ import annotations

import numpy as np

from .masks import pattern_matrix


def bf16_bits_to_f64(bits: np.ndarray) -> np.ndarray:
    """Exact widening of bf16 bit patterns (uint16) to fp64."""
    b = np.ascontiguousarray(bits, dtype=np.uint16)
    return (b.astype(np.uint32) << np.uint32(16)).view(np.float32).astype(np.float64)


def soft_choice(logits: np.ndarray, noise, tau: float) -> np.ndarray:
    """Eq. 3: z [G, 6] in fp64.  `noise` is the Gumbel sample per logit, or None for zeros."""
    s = np.asarray(logits, dtype=np.float64)
    assert s.ndim == 2 and s.shape[1] == 6 and tau > 0
    if noise is not None:
        s = s + np.asarray(noise, dtype=np.float64)
    s = s / float(tau)
    e = np.exp(s - s.max(axis=1, keepdims=True))  # the shift cancels in the quotient
    return e / e.sum(axis=1, keepdims=True)


def soft_block(z: np.ndarray) -> np.ndarray:
    """Eq. 2 with a relaxed z: b [G, 4] = (D z) per group."""
    D = pattern_matrix().astype(np.float64)  # 4 x 6
    return np.asarray(z, dtype=np.float64) @ D.T


def effective_weights(w_bits: np.ndarray, z: np.ndarray) -> np.ndarray:
    """Eq. 6 with the soft mask: W_eff in fp64 (unrounded), same shape as w_bits."""
    w = bf16_bits_to_f64(w_bits)
    return (soft_block(z) * w.reshape(-1, 4)).reshape(w.shape)


def logit_grad(z: np.ndarray, tau: float, w_bits: np.ndarray, g_w_eff: np.ndarray) -> np.ndarray:
    """dL/dlogits [G, 6] in fp64 from dL/dW_eff (any shape with 4 G elements in group order)."""
    z = np.asarray(z, dtype=np.float64)
    D = pattern_matrix().astype(np.float64)
    w = bf16_bits_to_f64(w_bits).reshape(-1, 4)
    g_b = np.asarray(g_w_eff, dtype=np.float64).reshape(-1, 4) * w
    g_z = g_b @ D  # [G, 6]: sum over the positions pattern i keeps
    inner = (z * g_z).sum(axis=1, keepdims=True)
    return z * (g_z - inner) / float(tau)


def conv_out_extent(size: int, k: int, stride: int, pad: int, dil: int) -> int:
    span = size + 2 * pad - dil * (k - 1) - 1
    return span // stride + 1 if span >= 0 else 0


def wgrad_f64(x_bits: np.ndarray, dy_bits: np.ndarray, KH: int, KW: int, stride: int, pad: int,
              dil: int) -> np.ndarray:
    """dL/dW_eff [C_out, KH, KW, C_in] in fp64 from x [N, H, W, C_in] and dL/dy [N, Ho, Wo, C_out]
    (both bf16 bit patterns, widened exactly).  One matrix product per filter tap over the
    zero-padded input; no other blocking."""
    x = bf16_bits_to_f64(x_bits)
    dy = bf16_bits_to_f64(dy_bits)
    N, H, W, C_in = x.shape
    Ho = conv_out_extent(H, KH, stride, pad, dil)
    Wo = conv_out_extent(W, KW, stride, pad, dil)
    assert dy.shape[:3] == (N, Ho, Wo), (dy.shape, (N, Ho, Wo))
    C_out = dy.shape[3]
    xp = np.zeros((N, H + 2 * pad, W + 2 * pad, C_in), dtype=np.float64)
    xp[:, pad:pad + H, pad:pad + W, :] = x
    dw = np.zeros((C_out, KH, KW, C_in), dtype=np.float64)
    dy2 = dy.reshape(-1, C_out)
    for kh in range(KH):
        for kw in range(KW):
            h0, w0 = kh * dil, kw * dil
            xs = xp[:, h0:h0 + stride * (Ho - 1) + 1:stride, w0:w0 + stride * (Wo - 1) + 1:stride, :]
            dw[:, kh, kw, :] = dy2.T @ xs.reshape(-1, C_in)
    return dw


def dgrad_f64(dy_bits: np.ndarray, w: np.ndarray, H: int, W: int, stride: int, pad: int, dil: int) -> np.ndarray:
    """dL/dx [N, H, W, C_in] in fp64 from dL/dy [N, Ho, Wo, C_out] (bf16 bit patterns) and weights
    [C_out, KH, KW, C_in] (fp64): every product x * w that enters y[n, ho, wo, co] hands dy * w back to
    that x (Eq. 4 differentiated in the input); one matrix product per filter tap, scattered to the
    input pixels the tap reads."""
    dy = bf16_bits_to_f64(dy_bits)
    w = np.asarray(w, dtype=np.float64)
    N, Ho, Wo, C_out = dy.shape
    _, KH, KW, C_in = w.shape
    dxp = np.zeros((N, H + 2 * pad, W + 2 * pad, C_in), dtype=np.float64)
    for kh in range(KH):
        for kw in range(KW):
            h0, w0 = kh * dil, kw * dil
            contrib = dy.reshape(-1, C_out) @ w[:, kh, kw, :]  # [N Ho Wo, C_in]
            dxp[:, h0:h0 + stride * (Ho - 1) + 1:stride, w0:w0 + stride * (Wo - 1) + 1:stride, :] += contrib.reshape(
                N, Ho, Wo, C_in)
    return dxp[:, pad:pad + H, pad:pad + W, :]


def adamw_step(theta, g, m, v, step: int, lr: float, beta1: float, beta2: float, eps: float, wd: float):
    """One AdamW update in fp64; `step` counts from 1.  Returns (theta, m, v) as new arrays."""
    theta = np.asarray(theta, dtype=np.float64)
    g = np.asarray(g, dtype=np.float64)
    m = beta1 * np.asarray(m, dtype=np.float64) + (1.0 - beta1) * g
    v = beta2 * np.asarray(v, dtype=np.float64) + (1.0 - beta2) * g * g
    mhat = m / (1.0 - beta1 ** step)
    vhat = v / (1.0 - beta2 ** step)
    theta = theta - lr * (mhat / (np.sqrt(vhat) + eps) + wd * theta)
    return theta, m, v
