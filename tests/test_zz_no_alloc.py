"""The entry point with built-in scratch, for hosts that may not allocate device memory.

Collected last on purpose (file name): a run that stops at the first failure has then already
run every other test.  The checks: two calls in a row through the C ABI agree with the regular entry
point (same inputs, caller-provided workspace) and with the fp64 oracle, within the tolerance the other
convolution tests use -- the second call matters because all calls share one scratch array that keeps
the previous call's contents; a call allocates nothing on the device; a layer too shallow to split and
layers beyond the entry point's limit behave as the header says.
"""
import pytest
import torch

from oracle import masks
from oracle.conv import conv2d_f64
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
    return inp, desc, x, w_comp, meta, b


def _oracle(inp):
    w_bits = synth.bf16_bits(inp.w)
    mask = masks.mask_from_pattern(parity.oracle_pattern(inp), w_bits.shape)
    return conv2d_f64(parity.oracle_shape(inp.spec), synth.bf16_bits(inp.x), w_bits, mask=mask, bias=inp.bias.numpy())


def test_static_scratch_entry_matches_regular_entry_and_oracle_twice():
    # deep K, few pixels: 8 output tiles, 36 weight tiles each -> the K range is split over 64 blocks
    spec = synth.LayerSpec("deepk_7x7", 8, 7, 7, 512, 512, 3, 3, 1, 1, 1, config=9, index=70)
    inp, desc, x, w_comp, meta, b = _prepared(spec)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    ref = api.ssconv_forward(desc, x, w_comp, meta, b, dev_status=status)
    torch.cuda.synchronize()
    ref64 = parity.bf16_tensor_to_f64(ref)
    want = _oracle(inp)
    for call in range(2):
        y = torch.full_like(ref, float("nan"))  # allocated by the test, not by the call
        api.ssconv_forward_static_ws(desc, x, w_comp, meta, b, y, dev_status=status)
        torch.cuda.synchronize()
        assert int(status.item()) == 0
        y64 = parity.bf16_tensor_to_f64(y)
        rel, mx = parity.errors(y64, ref64)
        assert rel <= parity.REL_FRO_TOL and mx <= parity.MAX_ABS_TOL, f"call {call} vs regular: rel={rel:.3e} max={mx:.3e}"
        rel, mx = parity.errors(y64, want)
        assert rel <= parity.REL_FRO_TOL and mx <= parity.MAX_ABS_TOL, f"call {call} vs oracle: rel={rel:.3e} max={mx:.3e}"


def test_static_scratch_entry_allocates_nothing():
    """After one warm call (module load, address look-up) a call changes neither torch's allocator
    statistics nor the device's free memory."""
    spec = synth.LayerSpec("deepk_small", 4, 7, 7, 256, 256, 3, 3, 1, 1, 1, config=9, index=72)
    inp, desc, x, w_comp, meta, b = _prepared(spec)
    y = torch.empty((spec.N, spec.H_out, spec.W_out, spec.C_out), dtype=torch.bfloat16, device=DEV)
    api.ssconv_forward_static_ws(desc, x, w_comp, meta, b, y)
    torch.cuda.synchronize()
    allocated, reserved = torch.cuda.memory_allocated(), torch.cuda.memory_reserved()
    free0, _ = torch.cuda.mem_get_info()
    for _ in range(3):
        api.ssconv_forward_static_ws(desc, x, w_comp, meta, b, y)
    torch.cuda.synchronize()
    free1, _ = torch.cuda.mem_get_info()
    assert torch.cuda.memory_allocated() == allocated and torch.cuda.memory_reserved() == reserved
    assert free1 == free0


def test_static_scratch_entry_on_a_layer_too_shallow_to_split():
    """One pair of k-blocks per tile: nothing to split, the scratch stays unused, the result is right."""
    spec = synth.LayerSpec("shallow_1x1", 2, 14, 14, 64, 128, 1, 1, 1, 0, 1, config=9, index=73)
    inp, desc, x, w_comp, meta, b = _prepared(spec)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    y = torch.full((spec.N, spec.H_out, spec.W_out, spec.C_out), float("nan"), dtype=torch.bfloat16, device=DEV)
    api.ssconv_forward_static_ws(desc, x, w_comp, meta, b, y, dev_status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    rel, mx = parity.errors(parity.bf16_tensor_to_f64(y), _oracle(inp))
    assert rel <= parity.REL_FRO_TOL and mx <= parity.MAX_ABS_TOL


def test_static_scratch_entry_limit_and_the_fallback_it_points_to():
    """64 output tiles are accepted, more are refused with SSCONV_ERR_UNSUPPORTED_SHAPE; for those the
    header points to ssconv_forward with ws = NULL, which must then work for any layer -- also a deep-K
    one above the limit, which ssconv_forward would split if it had a workspace."""
    at_limit = synth.LayerSpec("tiles_64", 1, 120, 128, 64, 64, 1, 1, 1, 0, 1, config=9, index=74)   # 15360 / 240 = 64
    inp, desc, x, w_comp, meta, b = _prepared(at_limit)
    y = torch.empty((1, 120, 128, 64), dtype=torch.bfloat16, device=DEV)
    api.ssconv_forward_static_ws(desc, x, w_comp, meta, b, y)
    torch.cuda.synchronize()
    rel, mx = parity.errors(parity.bf16_tensor_to_f64(y), _oracle(inp))
    assert rel <= parity.REL_FRO_TOL and mx <= parity.MAX_ABS_TOL

    # 1024 -> 256 channels, 3x3, 14x14 at batch 90: 74 x 2 = 148 output tiles of 144 k-blocks
    deep = synth.LayerSpec("deepk_over_limit", 90, 14, 14, 1024, 256, 3, 3, 1, 1, 1, config=9, index=75)
    inp, desc, x, w_comp, meta, b = _prepared(deep)
    y = torch.empty((deep.N, 14, 14, 256), dtype=torch.bfloat16, device=DEV)
    with pytest.raises(api.SsconvError) as e:
        api.ssconv_forward_static_ws(desc, x, w_comp, meta, b, y)
    assert e.value.status == 3
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    f = api.lib().ssconv_forward
    rc = f(api.ctypes.byref(desc), x.data_ptr(), w_comp.data_ptr(), meta.data_ptr(), b.data_ptr(), y.data_ptr(), None, 0,
           status.data_ptr(), None)
    torch.cuda.synchronize()
    assert rc == 0 and int(status.item()) == 0
    rng_idx = torch.randperm(y.numel())[:20000].numpy()
    w_bits = synth.bf16_bits(inp.w)
    mask = masks.mask_from_pattern(parity.oracle_pattern(inp), w_bits.shape)
    from oracle.conv import conv2d_f64_sample
    want = conv2d_f64_sample(parity.oracle_shape(deep), synth.bf16_bits(inp.x), w_bits, rng_idx, mask=mask, bias=inp.bias.numpy())
    rel, mx = parity.errors(parity.bf16_tensor_to_f64(y.reshape(-1)[torch.from_numpy(rng_idx)]), want)
    assert rel <= parity.REL_FRO_TOL and mx <= parity.MAX_ABS_TOL
