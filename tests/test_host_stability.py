"""The stability thresholds of Lemmas 3.4-3.6 are host arithmetic inside the library: checked against
the oracle without a GPU."""
import pytest

from oracle import stability
from paper_2411_00288_b200 import api


def test_thresholds_match_oracle():
    norms = [2.0, 0.5, 3.0, 1.25]
    for j in range(4):
        assert api.ssconv_stability_threshold(api.LEMMA_PERTURBATION, 1.5, norms, j, 0.3, 2.0) == pytest.approx(
            stability.threshold_perturbation(1.5, norms, j, 0.3, 2.0), rel=1e-13)
        assert api.ssconv_stability_threshold(api.LEMMA_ANY_MASK, 1.5, norms, j, 0.0, 2.0) == pytest.approx(
            stability.threshold_any_mask(1.5, norms, 2.0), rel=1e-13)
        assert api.ssconv_stability_threshold(api.LEMMA_MASKED_UPDATE, 1.5, norms, j, 0.7, 2.0) == pytest.approx(
            stability.threshold_masked_update(1.5, norms, j, 0.7, 2.0), rel=1e-13)
    with pytest.raises(ValueError):
        api.ssconv_stability_threshold(99, 1.0, norms, 0, 0.0, 1.0)
