"""A seeded random sweep of layer shapes against the fp64 oracle (Eq. 4 over the masked weights of Eq. 6):
shapes nobody picked by hand, so that the planner's tile widths, ragged channel tails, paddings, strides,
dilations and non-square filters meet in combinations the curated sweeps do not list.  Full tensors."""
import numpy as np
import pytest
import torch

from paper_2411_00288_b200 import synth
from tests import parity

pytestmark = pytest.mark.gpu
DEV = torch.device("cuda", 0)


def _draw_cases(count=40, seed=2411_00288):
    rng = np.random.default_rng(seed)
    cases = []
    while len(cases) < count:
        KH, KW = (int(rng.choice([1, 1, 2, 3, 3, 5, 7])) for _ in range(2))
        d = int(rng.choice([1, 1, 1, 2]))
        s = int(rng.choice([1, 1, 2, 3]))
        # the library refuses padding beyond the filter's extent
        p = int(rng.integers(0, min(d * (KH - 1), d * (KW - 1)) + 1)) if min(KH, KW) > 1 else 0
        N = int(rng.integers(1, 4))
        H, W = int(rng.integers(1, 41)), int(rng.integers(1, 41))
        Ci = int(rng.choice([8, 16, 24, 40, 64, 72, 96, 128, 136, 192, 256, 320]))
        Co = int(rng.choice([8, 16, 24, 40, 64, 72, 96, 128, 136, 200, 256, 264]))
        spec = synth.LayerSpec(f"rnd{len(cases)}", N, H, W, Ci, Co, KH, KW, s, p, d, relu=bool(rng.integers(0, 2)),
                               has_bias=bool(rng.integers(0, 4)), gelu=bool(rng.integers(0, 5) == 0),
                               mask_source=str(rng.choice(["magnitude", "gumbel_logits"])), config=12, index=len(cases))
        if spec.H_out < 1 or spec.W_out < 1 or spec.P * Co * spec.K > 6e8:
            continue
        cases.append((spec, bool(rng.integers(0, 3) == 0)))
    return cases


CASES = _draw_cases()


def _id(c):
    s = c[0]
    return (f"{s.name}_{s.N}x{s.H}x{s.W}x{s.C_in}to{s.C_out}_k{s.KH}x{s.KW}s{s.stride}p{s.pad}d{s.dil}"
            f"{'_gelu' if s.gelu else '_relu' if s.relu else ''}{'_res' if c[1] else ''}")


@pytest.mark.parametrize("case", CASES, ids=[_id(c) for c in CASES])
@pytest.mark.parametrize("sparse", [True, False], ids=["sparse", "dense"])
def test_random_shape_matches_oracle(case, sparse):
    spec, residual = case
    rel, mx = parity.check_layer(spec, DEV, sparse=sparse, residual=residual)
    assert rel <= parity.REL_FRO_TOL and mx <= parity.MAX_ABS_TOL, f"{_id(case)}: rel={rel:.3e} max={mx:.3e}"


def test_the_draw_is_varied():
    """The sweep is only worth its time if the draw really spreads: several filter sizes, strides,
    dilations, channel counts on both sides of one tile, residual and GELU cases."""
    specs = [c[0] for c in CASES]
    assert len({(s.KH, s.KW) for s in specs}) >= 10
    assert {1, 2, 3} <= {s.stride for s in specs} and {1, 2} <= {s.dil for s in specs}
    assert any(s.C_out > 128 for s in specs) and any(s.C_out < 64 for s in specs) and any(s.C_in % 64 for s in specs)
    assert any(c[1] for c in CASES) and any(s.gelu for s in specs) and any(not s.has_bias for s in specs)
    assert any(s.KH != s.KW for s in specs)
