"""CPU oracle for the stability quantities of Sec. 3.2: norms of a layer's weight matrix and of
the additive perturbation a mask induces, and the confidence thresholds of the lemmas.

TEST INFRASTRUCTURE, not a product path: only the tests, the smoke check and the benchmark's
CPU-baseline leg may import this module.  It shares no code with the CUDA library and imports
nothing from the package.  Everything is fp64 numpy.

What it restates:

* A masking B of W is the additive perturbation dW = mu(B, W) with W + dW = B .* W, i.e.
  dW = (B - 1) .* W: the dropped entries, negated (Lemma 3.3).  In the maximum-absolute-row-sum
  norm, ||dW||_inf <= ||W||_inf, with equality when a row of largest sum loses all of its mass.
* W is the row-major matrix in R^{C_out x K} of Eq. 5: a row is one output channel.
* Lemma 3.4: a classifier of depth d with L-Lipschitz activations stays stable on a sample x under
  a perturbation dW_j of layer j if its confidence exceeds L^d ||dW_j|| ||x|| prod_{i != j} ||W_i||.
* Lemma 3.5: for any masking of layer j the threshold L^d ||x|| prod_i ||W_i|| suffices.
* Lemma 3.6: a mask learned for W_j and applied to the updated weights W_j + U_j:
  L^d (||W_j||_inf + ||U_j||_inf) ||x||_inf prod_{i != j} ||W_i||_inf.
"""
from __future__ import annotations

import numpy as np

from .masks import mask_from_pattern
from .train import bf16_bits_to_f64


def row_sum_norms(w_bits: np.ndarray, pattern: np.ndarray):
    """(||W||_inf, ||(B - 1) .* W||_inf, ||B .* W||_inf) for bf16 weights [C_out, ...] (rows are
    output channels) and one 2:4 pattern per group of four."""
    w = np.abs(bf16_bits_to_f64(w_bits)).reshape(w_bits.shape[0], -1)
    keep = mask_from_pattern(pattern, w.shape).astype(np.float64)
    return (float(w.sum(axis=1).max()), float((w * (1.0 - keep)).sum(axis=1).max()),
            float((w * keep).sum(axis=1).max()))


def abs_max(x_bits: np.ndarray) -> float:
    """||x||_inf of a bf16 tensor."""
    return float(np.abs(bf16_bits_to_f64(x_bits)).max()) if x_bits.size else 0.0


def threshold_perturbation(L: float, norms, j: int, pert_norm: float, x_norm: float) -> float:
    """Lemma 3.4: L^d ||dW_j|| ||x|| prod_{i != j} ||W_i|| for the layer norms `norms` (d of them)."""
    norms = [float(v) for v in norms]
    others = 1.0
    for i, v in enumerate(norms):
        if i != j:
            others *= v
    return float(L) ** len(norms) * float(pert_norm) * float(x_norm) * others


def threshold_any_mask(L: float, norms, x_norm: float) -> float:
    """Lemma 3.5: L^d ||x|| prod_i ||W_i||."""
    prod = 1.0
    for v in norms:
        prod *= float(v)
    return float(L) ** len(list(norms)) * float(x_norm) * prod


def threshold_masked_update(L: float, norms, j: int, update_norm: float, x_norm: float) -> float:
    """Lemma 3.6: L^d (||W_j|| + ||U_j||) ||x|| prod_{i != j} ||W_i||."""
    norms = [float(v) for v in norms]
    return threshold_perturbation(L, norms, j, norms[j] + float(update_norm), x_norm)
