"""The entry point with built-in scratch, for hosts that may not allocate device memory.

Collected last on purpose (file name): a run that stops at the first failure has then already
run every other test.  The check: two calls in a row through the C ABI give what the regular
entry point gives (same inputs, caller-provided workspace), within the tolerance the other
convolution tests use.  The second call matters because all calls share one scratch array that
keeps the previous call's contents.
"""
import pytest
import torch

from paper_2411_00288_b200 import api, synth
from tests import parity

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _prepared(spec):
    inp = synth.make_inputs(spec)
    desc = api.desc_from_spec(spec)
    x, w, b = inp.x.to(DEV), inp.w.to(DEV), inp.bias.to(DEV)
    pat = api.ssconv_select_mask(api.MASK_MAGNITUDE_BF16, w, spec.G)
    w_comp, meta = api.ssconv_compress(desc, w, pat)
    return desc, x, w_comp, meta, b


def test_static_scratch_entry_matches_regular_entry_twice():
    # deep K, few pixels: 8 output tiles, 36 weight tiles each -> the K range is split over 64 blocks
    spec = synth.LayerSpec("deepk_7x7", 8, 7, 7, 512, 512, 3, 3, 1, 1, 1, config=9, index=70)
    desc, x, w_comp, meta, b = _prepared(spec)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    ref = api.ssconv_forward(desc, x, w_comp, meta, b, dev_status=status)
    torch.cuda.synchronize()
    ref64 = parity.bf16_tensor_to_f64(ref)
    for call in range(2):
        y = torch.full_like(ref, float("nan"))  # allocated by the test, not by the call
        api.ssconv_forward_static_ws(desc, x, w_comp, meta, b, y, dev_status=status)
        torch.cuda.synchronize()
        assert int(status.item()) == 0
        rel, mx = parity.errors(parity.bf16_tensor_to_f64(y), ref64)
        assert rel <= parity.REL_FRO_TOL and mx <= parity.MAX_ABS_TOL, f"call {call}: rel={rel:.3e} max={mx:.3e}"


def test_static_scratch_entry_rejects_layers_beyond_its_limit():
    # 56x56 at batch 4: 53 pixel tiles x 2 channel tiles = 106 output tiles > 64
    spec = synth.LayerSpec("too_big", 4, 56, 56, 64, 256, 1, 1, 1, 0, 1, config=9, index=71)
    desc, x, w_comp, meta, b = _prepared(spec)
    y = torch.empty((4, 56, 56, 256), dtype=torch.bfloat16, device=DEV)
    with pytest.raises(api.SsconvError) as e:
        api.ssconv_forward_static_ws(desc, x, w_comp, meta, b, y)
    assert e.value.status == 3
