"""GPU parity across the tile widths and partitions the host planner can choose.

The forward call picks, per layer, the number of positions per output tile (a multiple of 16 up to
240, so that the tiles fill the SMs) and whether the K range is split across thread blocks.  The
shapes below are sized so that, on a 148-SM device, the planner lands on widths from narrow to the
full 240, including widths whose last epilogue piece is short, and on a split plan; each is checked
against the fp64 oracle, and the test reports which plans were covered.
"""
import pytest
import torch

from paper_2411_00288_b200 import api, synth
from tests import parity

pytestmark = pytest.mark.gpu
DEV = "cuda:0"

# 3x3, 64 -> 64 channels, one image of H x W: the position count decides the tile width
SQUARES = [(84, 84), (119, 119), (128, 129), (137, 138), (161, 161), (175, 175), (188, 188)]
_seen = {}


@pytest.mark.parametrize("hw", SQUARES, ids=[f"{h}x{w}" for h, w in SQUARES])
@pytest.mark.parametrize("sparse", [True, False], ids=["sparse", "dense"])
def test_tile_width_sweep(hw, sparse):
    h, w = hw
    spec = synth.LayerSpec(f"tile_{h}x{w}", 1, h, w, 64, 64, 3, 3, 1, 1, 1, relu=True, w_std="fan_in",
                           mask_source="magnitude", config=8, index=SQUARES.index(hw))
    plan = api.ssconv_plan(api.desc_from_spec(spec), sparse)
    assert 48 <= plan["tile_positions"] <= 240 and plan["tile_positions"] % 16 == 0
    assert 2 <= plan["ring_groups"] <= 4 and plan["ctas"] >= 1
    _seen[(hw, sparse)] = plan
    rel, mx = parity.check_layer(spec, DEV, sparse=sparse, sample=20000)
    assert rel <= parity.REL_FRO_TOL and mx <= parity.MAX_ABS_TOL, f"{spec.name} {plan}: rel={rel:.3e} max={mx:.3e}"


def test_split_plan_deep_k_few_tiles():
    """512 -> 256 channels on 7x7 maps: few tiles, deep K: the K range is split and a second kernel finishes."""
    spec = synth.LayerSpec("split_7x7", 8, 7, 7, 512, 256, 3, 3, 1, 1, 1, relu=True, w_std="fan_in",
                           mask_source="magnitude", config=8, index=20)
    desc = api.desc_from_spec(spec)
    for sparse in (True, False):
        plan = api.ssconv_plan(desc, sparse)
        assert plan["split"], plan
        c0 = api.ssconv_launch_count()
        rel, mx = parity.check_layer(spec, DEV, sparse=sparse)
        assert rel <= parity.REL_FRO_TOL and mx <= parity.MAX_ABS_TOL, f"split {sparse}: rel={rel:.3e} max={mx:.3e}"
        rel, mx = parity.check_layer(spec, DEV, sparse=sparse, residual=True)  # the finishing kernel adds it
        assert rel <= parity.REL_FRO_TOL and mx <= parity.MAX_ABS_TOL, f"split+res {sparse}: rel={rel:.3e} max={mx:.3e}"
        assert api.ssconv_launch_count() - c0 >= 2  # main + finishing kernel (+ select/compress when sparse)


def test_zz_sweep_covered_several_widths():
    """Runs after the sweep (same file, later name): the planner must have used several distinct widths,
    at least one with a short last epilogue piece, and the widest."""
    if not _seen:
        pytest.skip("sweep did not run in this process")
    widths = {p["tile_positions"] for p in _seen.values()}
    assert len(widths) >= 4, widths
    assert any((bn // 2) % 40 != 0 for bn in widths), widths
    assert 240 in widths, widths
