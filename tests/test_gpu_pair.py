"""GPU parity of the pair kernel (tiles of 256 output channels on two thread blocks that share one
tensor-core instruction) against the fp64 oracle.

The planner uses the pair kernel for layers with more than 128 output channels when its cost model
prefers it; here it is forced on through ssconv_tune (and off, as the control) over shapes chosen to
hit its corners: an odd number of 128-channel tiles (the last pair's second block has no channels),
ragged output channels inside the second block, position tails, tiles narrower and wider than the
default, strides, dilation, channel tails, 1x1 and 3x3 filters, both weight forms, every activation.
"""
import pytest
import torch

from paper_2411_00288_b200 import api, synth
from tests import parity

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


@pytest.fixture(autouse=True)
def _reset_tuning():
    yield
    api.ssconv_tune(api.TUNE_PAIR, -1)
    api.ssconv_tune(api.TUNE_TILE_POSITIONS, 0)
    api.ssconv_tune(api.TUNE_PAIR_TILES, -1)


def _spec(name, n, h, w, cin, cout, k, stride, pad, dil=1, relu=True, gelu=False, idx=0):
    return synth.LayerSpec(name, n, h, w, cin, cout, k, k, stride, pad, dil, relu=relu, gelu=gelu, w_std="fan_in",
                           mask_source="magnitude", config=10, index=idx)


SHAPES = [
    _spec("pair_1x1_256", 4, 14, 14, 256, 256, 1, 1, 0, idx=0),
    _spec("pair_3x3_256", 4, 14, 14, 256, 256, 3, 1, 1, idx=1),
    _spec("pair_3x3_co384_odd_tiles", 2, 14, 14, 128, 384, 3, 1, 1, idx=2),
    _spec("pair_1x1_co200_ragged", 3, 17, 13, 64, 200, 1, 1, 0, idx=3),
    _spec("pair_1x1_co136", 3, 17, 13, 64, 136, 1, 1, 0, idx=4),              # 8 channels in the second block
    _spec("pair_3x3_s2_512", 2, 14, 14, 256, 512, 3, 2, 1, idx=5),
    _spec("pair_3x3_d2_p2", 2, 20, 20, 64, 256, 3, 1, 2, dil=2, idx=6),
    _spec("pair_1x1_tail_c96", 2, 28, 28, 96, 384, 1, 1, 0, idx=7),           # channel tail in the last chunk
    _spec("pair_1x1_c8", 2, 12, 12, 8, 256, 1, 1, 0, idx=8),                  # one partly filled k-block
    _spec("pair_1x1_odd_kblocks", 2, 12, 12, 192, 256, 1, 1, 0, idx=9),       # 3 k-blocks: the last group is half empty
    _spec("pair_3x3_norelu", 2, 14, 14, 128, 256, 3, 1, 1, relu=False, idx=10),
    _spec("pair_1x1_gelu", 2, 14, 14, 96, 384, 1, 1, 0, relu=False, gelu=True, idx=11),
    _spec("pair_7x7_wrap_2048", 8, 7, 7, 512, 2048, 1, 1, 0, idx=12),         # images wrap inside a tile; 8 pairs of tiles
]


@pytest.mark.parametrize("spec", SHAPES, ids=[s.name for s in SHAPES])
@pytest.mark.parametrize("sparse", [True, False], ids=["sparse", "dense"])
def test_pair_forced_matches_oracle(spec, sparse):
    if not sparse and spec.C_in == 8:
        pytest.skip("dense layers with 8 input channels run in the 8-channel mode of the one-block kernel")
    api.ssconv_tune(api.TUNE_PAIR, 1)
    plan = api.ssconv_plan(api.desc_from_spec(spec), sparse)
    assert plan["pair"] and plan["ctas"] % 2 == 0, plan
    rel, mx = parity.check_layer(spec, DEV, sparse=sparse)
    assert rel <= parity.REL_FRO_TOL and mx <= parity.MAX_ABS_TOL, f"{spec.name} {plan}: rel={rel:.3e} max={mx:.3e}"


@pytest.mark.parametrize("bn", [64, 80, 112, 176, 208, 240])
def test_pair_tile_widths(bn):
    """Forced tile widths, including ones whose last epilogue piece is short, on enough tiles that every
    pair works through several of them (ring and accumulator phases wrap)."""
    api.ssconv_tune(api.TUNE_PAIR, 1)
    api.ssconv_tune(api.TUNE_TILE_POSITIONS, bn)
    spec = _spec(f"pair_bn{bn}", 40, 28, 28, 128, 256, 1, 1, 0, idx=20)
    for sparse in (True, False):
        plan = api.ssconv_plan(api.desc_from_spec(spec), sparse)
        assert plan["pair"] and plan["tile_positions"] == bn, plan
        rel, mx = parity.check_layer(spec, DEV, sparse=sparse, sample=40000)
        assert rel <= parity.REL_FRO_TOL and mx <= parity.MAX_ABS_TOL, f"bn {bn} sparse={sparse}: rel={rel:.3e} max={mx:.3e}"


def test_pair_off_is_respected_and_narrow_layers_never_pair():
    spec = SHAPES[0]
    api.ssconv_tune(api.TUNE_PAIR, 0)
    assert not api.ssconv_plan(api.desc_from_spec(spec), True)["pair"]
    rel, mx = parity.check_layer(spec, DEV, sparse=True)
    assert rel <= parity.REL_FRO_TOL and mx <= parity.MAX_ABS_TOL
    api.ssconv_tune(api.TUNE_PAIR, 1)
    narrow = _spec("pair_not_128", 2, 14, 14, 128, 128, 1, 1, 0, idx=30)
    assert not api.ssconv_plan(api.desc_from_spec(narrow), True)["pair"]
    rel, mx = parity.check_layer(narrow, DEV, sparse=True)
    assert rel <= parity.REL_FRO_TOL and mx <= parity.MAX_ABS_TOL


def test_pair_output_guard_bands_and_determinism():
    """The output sits between sentinel bands that must stay untouched; two runs give the same bits."""
    api.ssconv_tune(api.TUNE_PAIR, 1)
    spec = _spec("pair_guard", 3, 13, 11, 64, 328, 3, 1, 1, idx=40)
    inp = synth.make_inputs(spec)
    desc = api.desc_from_spec(spec)
    w = inp.w.to(DEV)
    pat = api.ssconv_select_mask(api.MASK_MAGNITUDE_BF16, w, spec.G)
    w_comp, meta = api.ssconv_compress(desc, w, pat)
    n_out = spec.P * spec.C_out
    band = 4096
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    outs = []
    for _ in range(2):
        buf = torch.full((n_out + 2 * band,), -7.0, dtype=torch.bfloat16, device=DEV)
        y = buf[band:band + n_out].view(spec.N, spec.H_out, spec.W_out, spec.C_out)
        api.ssconv_forward(desc, inp.x.to(DEV), w_comp, meta, inp.bias.to(DEV), y=y, dev_status=status)
        torch.cuda.synchronize()
        assert int(status.item()) == 0
        assert bool((buf[:band] == -7.0).all()) and bool((buf[band + n_out:] == -7.0).all())
        assert bool((y >= 0).all())  # ReLU output: every element was written
        outs.append(y.clone())
    assert torch.equal(outs[0], outs[1])


# ---- two position tiles per work item (the pair's ring group holds the weights once for both)
@pytest.mark.parametrize("spec", SHAPES, ids=[s.name for s in SHAPES])
@pytest.mark.parametrize("sparse", [True, False], ids=["sparse", "dense"])
def test_pair_with_two_tiles_per_item_forced_matches_oracle(spec, sparse):
    """The same corner shapes with two tiles per work item forced on: odd numbers of position tiles (the last
    item's second tile lies past the last position: it reads zeros and stores nothing), items whose tiles wrap
    images, ragged channels, every activation, both weight forms."""
    if not sparse and spec.C_in == 8:
        pytest.skip("dense layers with 8 input channels run in the 8-channel mode of the one-block kernel")
    api.ssconv_tune(api.TUNE_PAIR, 1)
    api.ssconv_tune(api.TUNE_PAIR_TILES, 1)
    api.ssconv_tune(api.TUNE_TILE_POSITIONS, 112 if spec.index % 2 else 176)
    plan = api.ssconv_plan(api.desc_from_spec(spec), sparse)
    assert plan["pair"], plan
    rel, mx = parity.check_layer(spec, DEV, sparse=sparse)
    assert rel <= parity.REL_FRO_TOL and mx <= parity.MAX_ABS_TOL, f"{spec.name} {plan}: rel={rel:.3e} max={mx:.3e}"


@pytest.mark.parametrize("bn", [64, 96, 144, 192])
def test_pair_with_two_tiles_per_item_over_many_items(bn):
    """Every pair works through several items (ring and accumulator phases wrap), at tile widths whose last
    epilogue piece is short, with an odd and an even number of position tiles; bit for bit what the
    one-tile-per-item form gives (same products, same order per tile)."""
    for n in (40, 41):
        spec = _spec(f"dual_bn{bn}_{n}", n, 28, 28, 128, 256, 3, 1, 1, idx=30 + n)
        inp = synth.make_inputs(spec)
        desc = api.desc_from_spec(spec)
        x, w, bias = inp.x.to(DEV), inp.w.to(DEV), inp.bias.to(DEV)
        pat = api.ssconv_select_mask(api.MASK_MAGNITUDE_BF16, w, spec.G)
        w_comp, meta = api.ssconv_compress(desc, w, pat)
        status = torch.zeros(1, dtype=torch.int32, device=DEV)
        api.ssconv_tune(api.TUNE_PAIR, 1)
        api.ssconv_tune(api.TUNE_TILE_POSITIONS, bn)
        outs = []
        for tiles in (0, 1):
            api.ssconv_tune(api.TUNE_PAIR_TILES, tiles)
            outs.append(api.ssconv_forward(desc, x, w_comp, meta, bias, dev_status=status))
        torch.cuda.synchronize()
        assert int(status.item()) == 0
        assert torch.equal(outs[0], outs[1])
        rel, mx = parity.check_layer(spec, DEV, sparse=True, sample=30000)
        assert rel <= parity.REL_FRO_TOL and mx <= parity.MAX_ABS_TOL, f"bn {bn} n {n}: rel={rel:.3e} max={mx:.3e}"


def test_two_tiles_per_item_is_the_planners_choice_only_where_it_was_measured_to_pay():
    """Deep K, two or more pairs of channel tiles, about one item per pair: yes (ResNet-50's last stage at batch
    256); one pair of channel tiles, a shallow K, few items or the dense form: no.  The call must then agree with
    the same layer run one tile per item."""
    yes = synth.LayerSpec("s4_3x3", 256, 7, 7, 512, 512, 3, 3, 1, 1, 1, config=10, index=50)
    d = api.desc_from_spec(yes)
    auto = api.ssconv_plan(d, True)
    api.ssconv_tune(api.TUNE_PAIR_TILES, 0)
    single = api.ssconv_plan(d, True)
    api.ssconv_tune(api.TUNE_PAIR_TILES, -1)
    assert auto["pair"] and single["pair"] and auto["tile_positions"] == single["tile_positions"]
    assert auto["ctas"] == 144 and single["ctas"] == 148, (auto, single)     # 72 items of two tiles against 144 tiles
    assert api.ssconv_plan(d, False)["ctas"] == 148                           # the dense form: one tile per item
    for n, h, ci, co, k in ((256, 14, 256, 256, 3), (256, 14, 1024, 512, 1), (64, 7, 512, 512, 3), (256, 7, 2048, 512, 1)):
        dn = api.make_desc(n, h, h, ci, co, k, k, 1, k // 2)
        a = api.ssconv_plan(dn, True)
        api.ssconv_tune(api.TUNE_PAIR_TILES, 0)
        b = api.ssconv_plan(dn, True)
        api.ssconv_tune(api.TUNE_PAIR_TILES, -1)
        assert a == b, (a, b)
    rel, mx = parity.check_layer(yes, DEV, sparse=True, sample=30000)
    assert rel <= parity.REL_FRO_TOL and mx <= parity.MAX_ABS_TOL


# ---- the fused skip connection on pairs
RES_SHAPES = [SHAPES[i] for i in (1, 2, 3, 5, 7, 9, 11, 12)]


@pytest.mark.parametrize("spec", RES_SHAPES, ids=[s.name for s in RES_SHAPES])
@pytest.mark.parametrize("sparse", [True, False], ids=["sparse", "dense"])
def test_pair_forced_with_residual_matches_oracle(spec, sparse):
    """y = act(bias + conv + residual) on thread-block pairs: residual pieces prefetched into four staging
    buffers per group by each block for its own channels; odd numbers of channel tiles (a block without
    channels only keeps its barriers in step), ragged channels, short last pieces, GELU."""
    api.ssconv_tune(api.TUNE_PAIR, 1)
    rel, mx = parity.check_layer(spec, DEV, sparse=sparse, residual=True)
    assert rel <= parity.REL_FRO_TOL and mx <= parity.MAX_ABS_TOL, f"{spec.name}: rel={rel:.3e} max={mx:.3e}"


@pytest.mark.parametrize("bn", [64, 112, 176, 208])
def test_pair_with_residual_over_many_tiles_and_in_place(bn):
    """Several tiles per pair (staging buffers and their barriers wrap many times), the residual read from the
    output's own buffer, against the same call on one-block tiles bit for bit (same products, same order)."""
    spec = _spec(f"pair_res_bn{bn}", 24, 28, 28, 256, 512, 1, 1, 0, idx=60)
    inp = synth.make_inputs(spec)
    desc = api.desc_from_spec(spec)
    x, w, bias = inp.x.to(DEV), inp.w.to(DEV), inp.bias.to(DEV)
    pat = api.ssconv_select_mask(api.MASK_MAGNITUDE_BF16, w, spec.G)
    w_comp, meta = api.ssconv_compress(desc, w, pat)
    res = parity.make_residual(spec, None).to(DEV)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    outs = []
    for pair in (0, 1):
        api.ssconv_tune(api.TUNE_PAIR, pair)
        api.ssconv_tune(api.TUNE_TILE_POSITIONS, bn)
        y = res.clone()                       # in place: the residual is y's own buffer
        api.ssconv_forward(desc, x, w_comp, meta, bias, y=y, dev_status=status, residual=y)
        outs.append(y)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    assert torch.equal(outs[0], outs[1])
    api.ssconv_tune(api.TUNE_PAIR, 1)
    rel, mx = parity.check_layer(spec, DEV, sparse=True, sample=30000, residual=True)
    assert rel <= parity.REL_FRO_TOL and mx <= parity.MAX_ABS_TOL, f"bn {bn}: rel={rel:.3e} max={mx:.3e}"
