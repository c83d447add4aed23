"""Pins for the stability oracle (CPU only): the norms against numpy's matrix-norm routine and
closed forms, Lemma 3.3's bound and its tight case, and the lemmas' thresholds against each other."""
import numpy as np
import pytest

from oracle import masks, stability
from tests.brute import bf16_to_f64, f32_to_bf16_bits


def _bits(rng, shape, scale=1.0):
    return f32_to_bf16_bits((rng.normal(size=shape) * scale).astype(np.float32))


def test_norms_match_the_library_matrix_norm_of_the_three_matrices():
    rng = np.random.default_rng(21)
    w = _bits(rng, (24, 3, 3, 16))
    pat = masks.select_from_magnitude(w)
    full, dropped, kept = stability.row_sum_norms(w, pat)
    W = bf16_to_f64(w).reshape(24, -1)
    B = masks.mask_from_pattern(pat, W.shape).astype(np.float64)
    assert full == pytest.approx(np.linalg.norm(W, np.inf), rel=1e-14)
    assert dropped == pytest.approx(np.linalg.norm((B - 1.0) * W, np.inf), rel=1e-14)
    assert kept == pytest.approx(np.linalg.norm(B * W, np.inf), rel=1e-14)
    # W + dW = B .* W with dW = (B - 1) .* W  (Lemma 3.3's construction)
    np.testing.assert_array_equal(W + (B - 1.0) * W, B * W)


def test_closed_forms():
    w = np.full((5, 1, 1, 32), 0x3F80, dtype=np.uint16)  # all ones
    pat = np.zeros(5 * 8, dtype=np.uint8)
    assert stability.row_sum_norms(w, pat) == (32.0, 16.0, 16.0)
    w[3, 0, 0, :] = 0x4000  # one row of twos
    assert stability.row_sum_norms(w, pat) == (64.0, 32.0, 32.0)
    assert stability.abs_max(np.array([0x3F80, 0xC040, 0x0000], dtype=np.uint16)) == 3.0


def test_lemma_3_3_bound_holds_and_is_tight():
    rng = np.random.default_rng(22)
    for _ in range(20):
        w = _bits(rng, (8, 1, 1, 16))
        pat = rng.integers(0, 6, size=8 * 4).astype(np.uint8)
        full, dropped, kept = stability.row_sum_norms(w, pat)
        assert dropped <= full and kept <= full
        assert full <= dropped + kept + 1e-12
    # tight: the kept positions of every group hold zeros, so the mask removes all of W's mass
    w = np.zeros((2, 1, 1, 8), dtype=np.uint16)
    w[:, 0, 0, 2::4] = 0x3F80
    w[:, 0, 0, 3::4] = 0x4000
    full, dropped, kept = stability.row_sum_norms(w, np.zeros(4, dtype=np.uint8))  # pattern 0 keeps {0, 1}
    assert (full, dropped, kept) == (6.0, 6.0, 0.0)


def test_magnitude_masks_drop_at_most_half_of_each_rows_mass():
    rng = np.random.default_rng(23)
    w = _bits(rng, (16, 3, 3, 8))
    full, dropped, kept = stability.row_sum_norms(w, masks.select_from_magnitude(w))
    assert dropped <= 0.5 * full and kept >= 0.5 * full


def test_thresholds_follow_the_lemmas():
    norms = [2.0, 0.5, 3.0]
    # Lemma 3.4 with unit norms elsewhere
    assert stability.threshold_perturbation(1.0, [1.0, 1.0, 1.0], 1, 0.25, 4.0) == 1.0
    assert stability.threshold_perturbation(2.0, norms, 1, 0.1, 1.5) == pytest.approx(8.0 * 0.1 * 1.5 * 6.0)
    # Lemma 3.5 is Lemma 3.4 with the perturbation at its largest, ||dW_j|| = ||W_j|| (Lemma 3.3)
    assert stability.threshold_any_mask(2.0, norms, 1.5) == pytest.approx(
        stability.threshold_perturbation(2.0, norms, 1, norms[1], 1.5))
    for j in range(3):
        assert stability.threshold_perturbation(1.0, norms, j, 0.9 * norms[j], 1.0) < stability.threshold_any_mask(
            1.0, norms, 1.0)
    # Lemma 3.6 adds the update's norm to the masked layer's
    assert stability.threshold_masked_update(1.0, norms, 2, 0.5, 2.0) == pytest.approx((3.0 + 0.5) * 2.0 * 1.0)
    assert stability.threshold_masked_update(1.0, norms, 2, 0.0, 2.0) == pytest.approx(
        stability.threshold_any_mask(1.0, norms, 2.0))
