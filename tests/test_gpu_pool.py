"""Max-pooling on the GPU, bit-exact against a numpy maximum over the windows written from the definition
(padding never wins), on the 3 x 3 stride-2 form the ResNet stacks use (odd and even extents, several
strips of output rows, a single column of windows) and on other windows."""
import numpy as np
import pytest
import torch

from paper_2411_00288_b200 import api, synth

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _maxpool_numpy(x, k, s, p):
    N, H, W, C = x.shape
    Ho, Wo = (H + 2 * p - k) // s + 1, (W + 2 * p - k) // s + 1
    y = np.full((N, Ho, Wo, C), -np.inf, dtype=np.float32)
    for ho in range(Ho):
        for wo in range(Wo):
            h0, w0 = max(ho * s - p, 0), max(wo * s - p, 0)
            h1, w1 = min(ho * s - p + k, H), min(wo * s - p + k, W)
            y[:, ho, wo, :] = x[:, h0:h1, w0:w1, :].max(axis=(1, 2))
    return y


@pytest.mark.parametrize("shape,k,s,p", [
    ((2, 7, 9, 8), 3, 2, 1), ((3, 12, 12, 64), 3, 2, 1), ((1, 40, 6, 8), 3, 2, 1), ((2, 35, 3, 16), 3, 2, 1),
    ((1, 2, 2, 8), 3, 2, 1), ((4, 112, 112, 64), 3, 2, 1), ((2, 8, 8, 8), 2, 2, 0), ((1, 9, 7, 24), 3, 1, 1),
    ((1, 6, 10, 8), 5, 3, 2),
])
def test_maxpool_is_bit_exact(shape, k, s, p):
    g = torch.Generator().manual_seed(synth.SEED_BASE + 3600 + shape[1] + k)
    x = torch.randn(shape, generator=g).to(torch.bfloat16)
    Ho, Wo = api.ssconv_window_extent(shape[1], k, s, p), api.ssconv_window_extent(shape[2], k, s, p)
    band = 64
    buf = torch.full((shape[0] * Ho * Wo * shape[3] + 2 * band,), 9.0, dtype=torch.bfloat16, device=DEV)
    y = buf[band:-band].view(shape[0], Ho, Wo, shape[3])
    api.ssconv_maxpool(x.to(DEV), k, s, p, y=y)
    torch.cuda.synchronize()
    ref = _maxpool_numpy(x.float().numpy(), k, s, p)
    np.testing.assert_array_equal(y.float().cpu().numpy(), ref)
    assert bool((buf[:band] == 9.0).all()) and bool((buf[-band:] == 9.0).all())
