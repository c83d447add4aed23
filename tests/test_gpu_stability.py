"""GPU parity of the stability quantities of Sec. 3.2 (row-sum norms of W, of the mask's perturbation
and of the masked weights; ||x||_inf; the lemmas' thresholds) against the fp64 oracle."""
import numpy as np
import pytest
import torch

from oracle import masks, stability
from paper_2411_00288_b200 import api, synth

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
NORM_RTOL = 1e-5  # fp32 sums of up to 4608 exact bf16 magnitudes per row


@pytest.mark.parametrize("shape", [(8, 1, 1, 8), (64, 3, 3, 64), (136, 1, 1, 96), (512, 3, 3, 512), (3, 5, 5, 4)])
@pytest.mark.parametrize("source", ["magnitude", "random"])
def test_mask_norms_match_oracle(shape, source):
    g = torch.Generator().manual_seed(synth.SEED_BASE + 5100 + shape[0] + shape[3])
    w = (torch.randn(shape, generator=g) * 0.1).to(torch.bfloat16)
    G = w.numel() // 4
    if source == "magnitude":
        pat = masks.select_from_magnitude(synth.bf16_bits(w))
    else:
        pat = torch.randint(0, 6, (G,), generator=g).numpy().astype(np.uint8)
    out = api.ssconv_mask_norms(w.to(DEV), torch.from_numpy(pat).to(DEV)).cpu().numpy().astype(np.float64)
    ref = np.array(stability.row_sum_norms(synth.bf16_bits(w), pat))
    np.testing.assert_allclose(out, ref, rtol=NORM_RTOL)
    assert out[1] <= out[0] * (1 + NORM_RTOL)  # Lemma 3.3
    if source == "magnitude":
        assert out[1] <= 0.5 * out[0] * (1 + NORM_RTOL)


def test_mask_norms_are_recomputed_on_every_call():
    w = torch.ones((4, 1, 1, 8), dtype=torch.bfloat16, device=DEV)
    pat = torch.zeros((8,), dtype=torch.uint8, device=DEV)
    out = torch.full((3,), 123.0, dtype=torch.float32, device=DEV)
    api.ssconv_mask_norms(w, pat, out=out)
    assert out.cpu().tolist() == [8.0, 4.0, 4.0]
    api.ssconv_mask_norms(w * 0.5, pat, out=out)
    assert out.cpu().tolist() == [4.0, 2.0, 2.0]


@pytest.mark.parametrize("n", [0, 1, 7, 8, 4099, 1 << 22])
def test_absmax_is_exact(n):
    g = torch.Generator().manual_seed(77 + n)
    x = torch.randn((max(n, 1),), generator=g).to(torch.bfloat16)[:n].contiguous()
    if n > 3:
        x[n // 2] = -37.5
    got = float(api.ssconv_absmax(x.to(DEV) if n else torch.empty((0,), dtype=torch.bfloat16, device=DEV)).item())
    assert got == stability.abs_max(synth.bf16_bits(x))
