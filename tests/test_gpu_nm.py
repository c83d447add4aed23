"""General N:M masks on the GPU: selection and application bit-exact against the oracle, and a layer
masked 1:4 / 2:8 / 3:4 run through the dense kernel against the fp64 oracle of the masked convolution."""
import math

import numpy as np
import pytest
import torch

from oracle import masks
from oracle.conv import conv2d_f64
from paper_2411_00288_b200 import api, synth
from tests import parity

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
CASES = [(2, 4), (1, 4), (3, 4), (1, 2), (2, 8), (4, 8), (7, 8)]


@pytest.mark.parametrize("N,M", CASES)
def test_nm_selection_and_application_bit_exact(N, M):
    n = math.comb(M, N)
    assert api.ssconv_nm_patterns(N, M) == n
    rng = np.random.default_rng(31 * N + M)
    G = 5000
    w = torch.randn((G, M), generator=torch.Generator().manual_seed(N * 100 + M), dtype=torch.float32).to(torch.bfloat16)
    w[:200] = w[:200].abs().round()            # small integers: many equal magnitudes, mixed with zeros
    w[200:300, 1] = -w[200:300, 0]             # equal magnitudes, opposite signs
    bits = synth.bf16_bits(w)
    pat = api.ssconv_select_mask_nm(api.MASK_MAGNITUDE_BF16, w.to(DEV), G, N, M).cpu().numpy()
    want = masks.nm_select_from_magnitude((bits & 0x7FFF).astype(np.int64), N)
    assert np.array_equal(pat, want)
    scores = rng.normal(size=(G, n)).astype(np.float32)
    scores[:100, : min(n, 3)] = 1.5            # ties for the maximum: the first wins
    pl = api.ssconv_select_mask_nm(api.MASK_LOGITS_F32, torch.from_numpy(scores).to(DEV), G, N, M).cpu().numpy()
    assert np.array_equal(pl, masks.nm_select_from_logits(scores))
    masked = api.ssconv_apply_mask_nm(w.to(DEV), torch.from_numpy(want).to(DEV), N, M).cpu()
    m = masks.nm_mask_from_pattern(want, N, M, (G, M))
    assert np.array_equal(synth.bf16_bits(masked), np.where(m == 1, bits, 0).astype(np.uint16))


def test_nm_argument_rules():
    assert api.ssconv_nm_patterns(0, 4) == 0 and api.ssconv_nm_patterns(5, 4) == 0 and api.ssconv_nm_patterns(4, 9) == 0
    w = torch.zeros((8, 4), dtype=torch.bfloat16, device=DEV)
    with pytest.raises(api.SsconvError):
        api.ssconv_select_mask_nm(api.MASK_MAGNITUDE_BF16, w, 8, 5, 4)


@pytest.mark.parametrize("N,M", [(1, 4), (2, 8), (3, 4)])
def test_nm_masked_layer_through_the_dense_kernel_matches_oracle(N, M):
    spec = synth.LayerSpec(f"nm_{N}of{M}", 2, 14, 14, 64, 72, 3, 3, 1, 1, 1, relu=True, w_std="fan_in",
                           config=12, index=10 * N + M)
    inp = synth.make_inputs(spec)   # fan-in weights: outputs of order one, where the gates below are stated
    G = inp.w.numel() // M
    wd = inp.w.to(DEV)
    pat = api.ssconv_select_mask_nm(api.MASK_MAGNITUDE_BF16, wd, G, N, M)
    w_masked = api.ssconv_apply_mask_nm(wd, pat, N, M)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    y = api.ssconv_forward_dense(api.desc_from_spec(spec), inp.x.to(DEV), w_masked, inp.bias.to(DEV), dev_status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    bits = synth.bf16_bits(inp.w)
    want_pat = masks.nm_select_from_magnitude((bits.reshape(-1, M) & 0x7FFF).astype(np.int64), N)
    assert np.array_equal(pat.cpu().numpy(), want_pat)
    mask = masks.nm_mask_from_pattern(want_pat, N, M, bits.shape)
    assert mask.reshape(-1, M).sum(axis=1).tolist() == [N] * G
    ref = conv2d_f64(parity.oracle_shape(spec), synth.bf16_bits(inp.x), bits, mask=mask, bias=inp.bias.numpy())
    rel, mx = parity.errors(parity.bf16_tensor_to_f64(y), ref)
    assert rel <= parity.REL_FRO_TOL and mx <= parity.MAX_ABS_TOL, f"rel={rel:.3e} max={mx:.3e}"
