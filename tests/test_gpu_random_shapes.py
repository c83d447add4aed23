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


# ---------------------------------------------------------------- the training kernels on drawn shapes
def _draw_train_cases(count, seed, max_macs):
    rng = np.random.default_rng(seed)
    cases = []
    while len(cases) < count:
        KH, KW = (int(rng.choice([1, 1, 2, 3, 3, 5, 7])) for _ in range(2))
        d = int(rng.choice([1, 1, 1, 2]))
        s = int(rng.choice([1, 1, 2, 2, 3]))
        p = int(rng.integers(0, min(d * (KH - 1), d * (KW - 1)) + 1)) if min(KH, KW) > 1 else 0
        N, H, W = int(rng.integers(1, 5)), int(rng.integers(1, 33)), int(rng.integers(1, 33))
        Ci = int(rng.choice([8, 16, 40, 64, 72, 104, 128, 192, 256, 320]))
        Co = int(rng.choice([8, 24, 40, 64, 96, 128, 136, 200, 256, 328]))
        spec = synth.LayerSpec(f"trn{len(cases)}", N, H, W, Ci, Co, KH, KW, s, p, d, config=13, index=len(cases))
        if spec.H_out < 1 or spec.W_out < 1 or spec.P * Co * spec.K > max_macs:
            continue
        cases.append(spec)
    return cases


def _tid(s):
    return f"{s.name}_{s.N}x{s.H}x{s.W}x{s.C_in}to{s.C_out}_k{s.KH}x{s.KW}s{s.stride}p{s.pad}d{s.dil}"


WG_CASES = _draw_train_cases(24, 2411_00289, 4e8)
DG_CASES = _draw_train_cases(24, 2411_00290, 2e8)


@pytest.mark.parametrize("spec", WG_CASES, ids=[_tid(s) for s in WG_CASES])
def test_random_shape_weight_gradient_matches_oracle(spec):
    """dL/dW of Eq. 4 (Sec. 3.1's training step differentiates it): fp32 accumulation of exact products."""
    from oracle import train as otrain
    from paper_2411_00288_b200 import api
    inp = synth.make_inputs(spec, x_only=True)
    tr = synth.make_train_inputs(spec)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    dw = api.ssconv_wgrad(api.desc_from_spec(spec), inp.x.to(DEV), tr.dy.to(DEV), dev_status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    ref = otrain.wgrad_f64(synth.bf16_bits(inp.x), synth.bf16_bits(tr.dy), spec.KH, spec.KW, spec.stride, spec.pad,
                           spec.dil)
    got = dw.cpu().numpy().astype(np.float64)
    assert got.shape == ref.shape
    scale = max(float(np.abs(ref).max()), 1e-30)
    rel = float(np.linalg.norm(got - ref) / max(np.linalg.norm(ref), 1e-30))
    assert rel <= 1e-4 and float(np.abs(got - ref).max()) <= 2e-4 * scale, (_tid(spec), rel)


@pytest.mark.parametrize("spec", DG_CASES, ids=[_tid(s) for s in DG_CASES])
def test_random_shape_input_gradient_matches_oracle(spec):
    """dL/dx of Eq. 4 in one call (residue classes of the input position for strided layers), with sentinel
    bands around the gradient and the workspace."""
    from oracle import train as otrain
    from paper_2411_00288_b200 import api
    g = torch.Generator().manual_seed(synth.SEED_BASE + 5200 + spec.index)
    w = (torch.randn((spec.C_out, spec.KH, spec.KW, spec.C_in), generator=g) * (2.0 / spec.K) ** 0.5).to(torch.bfloat16)
    dy = torch.randn((spec.N, spec.H_out, spec.W_out, spec.C_out), generator=g).to(torch.bfloat16)
    desc = api.make_desc(spec.N, spec.H, spec.W, spec.C_in, spec.C_out, spec.KH, spec.KW, stride=spec.stride, pad=spec.pad,
                         dil=spec.dil)
    band = 2048
    n_dx = spec.N * spec.H * spec.W * spec.C_in
    buf = torch.full((n_dx + 2 * band,), -7.0, dtype=torch.bfloat16, device=DEV)
    dx = buf[band:band + n_dx].view(spec.N, spec.H, spec.W, spec.C_in)
    need = api.ssconv_dgrad_ws_bytes(desc)
    wsbuf = torch.full((need + 2 * band,), 0x5A, dtype=torch.uint8, device=DEV)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    api.ssconv_dgrad(desc, dy.to(DEV), w.to(DEV), dx=dx, ws=wsbuf[band:band + need], dev_status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    assert bool((buf[:band] == -7.0).all()) and bool((buf[-band:] == -7.0).all())
    assert bool((wsbuf[:band] == 0x5A).all()) and bool((wsbuf[-band:] == 0x5A).all())
    ref = otrain.dgrad_f64(synth.bf16_bits(dy), parity.bf16_tensor_to_f64(w), spec.H, spec.W, spec.stride, spec.pad, spec.dil)
    rel, mx = parity.errors(parity.bf16_tensor_to_f64(dx), ref)
    assert rel <= parity.REL_FRO_TOL and mx <= parity.MAX_ABS_TOL * max(1.0, float(np.abs(ref).max()) / 4.0), (_tid(spec), rel, mx)


# ---------------------------------------------------------------- pooling, depthwise convolution, layer norm
def _draw_block_cases(count, seed):
    rng = np.random.default_rng(seed)
    out = []
    while len(out) < count:
        K = int(rng.choice([2, 3, 3, 5, 7, 7]))
        s = int(rng.choice([1, 1, 1, 2, 3]))
        d = int(rng.choice([1, 1, 1, 2]))
        p = int(rng.integers(0, (K - 1) * d + 1))
        N, H, W = int(rng.integers(1, 4)), int(rng.integers(1, 30)), int(rng.integers(1, 30))
        C = int(rng.choice([8, 24, 32, 40, 64, 96, 160, 192, 200, 384]))
        if H + 2 * p < d * (K - 1) + 1 or W + 2 * p < d * (K - 1) + 1:
            continue
        out.append((N, H, W, C, K, s, p, d))
    return out


DW_CASES = _draw_block_cases(30, 2411_00292)


@pytest.mark.parametrize("case", DW_CASES, ids=[f"dw{i}_" + "x".join(map(str, c[:4])) + f"_k{c[4]}s{c[5]}p{c[6]}d{c[7]}"
                                                 for i, c in enumerate(DW_CASES)])
def test_random_shape_depthwise_matches_oracle(case):
    """Channel counts on both sides of the tile kernel's rule (multiples of 32), filters with and without a
    specialised kernel, strides and dilations (the generic kernel), maps smaller than one tile."""
    from oracle import blocks
    from oracle.conv import ConvShape
    from paper_2411_00288_b200 import api
    N, H, W, C, K, s, p, d = case
    g = torch.Generator().manual_seed(synth.SEED_BASE + 5300 + DW_CASES.index(case))
    x = torch.randn((N, H, W, C), generator=g).to(torch.bfloat16)
    w = (torch.randn((K, K, C), generator=g) / K).to(torch.bfloat16)
    bias = torch.randn((C,), generator=g) * 0.1
    relu = bool(DW_CASES.index(case) % 3 == 0)
    desc = api.make_desc(N, H, W, C, C, K, K, s, p, d, bias=True, relu=relu)
    Ho, Wo = api.ssconv_out_shape(desc)
    band = 256
    buf = torch.full((N * Ho * Wo * C + 2 * band,), -5.0, dtype=torch.bfloat16, device=DEV)
    y = buf[band:band + N * Ho * Wo * C].view(N, Ho, Wo, C)
    api.ssconv_depthwise(desc, x.to(DEV), w.to(DEV), bias.to(DEV), y=y)
    torch.cuda.synchronize()
    assert bool((buf[:band] == -5.0).all()) and bool((buf[-band:] == -5.0).all())
    shape = ConvShape(N, H, W, C, C, K, K, (s, s), (p, p), (d, d), relu=False)
    ref = blocks.depthwise_conv2d_f64(shape, synth.bf16_bits(x), synth.bf16_bits(w), bias=bias.numpy())
    if relu:
        ref = np.maximum(ref, 0.0)
    rel, mx = parity.errors(parity.bf16_tensor_to_f64(y), ref)
    assert rel <= parity.REL_FRO_TOL and mx <= parity.MAX_ABS_TOL, (case, rel, mx)


@pytest.mark.parametrize("pixels,C", [(1, 8), (37, 24), (301, 40), (77, 96), (64, 104), (129, 192), (50, 264), (33, 384),
                                      (19, 768), (7, 1024), (11, 1032), (23, 20), (5, 1048)])
def test_layernorm_over_channel_counts_matches_oracle(pixels, C):
    """Every lane grouping of the vector kernel (1 to 32 lanes per pixel, one to four pieces per lane, idle lanes
    and none), a pixel count that leaves a warp partly filled, and channel counts only the scalar kernel takes."""
    from oracle import blocks
    from paper_2411_00288_b200 import api
    g = torch.Generator().manual_seed(synth.SEED_BASE + 5400 + C)
    x = (torch.randn((pixels, C), generator=g) * 2 + 0.5).to(torch.bfloat16)
    gamma, beta = torch.randn((C,), generator=g) * 0.5 + 1.0, torch.randn((C,), generator=g) * 0.2
    band = 128
    buf = torch.full((pixels * C + 2 * band,), -5.0, dtype=torch.bfloat16, device=DEV)
    y = buf[band:band + pixels * C].view(pixels, C)
    api.ssconv_layernorm(x.to(DEV), gamma.to(DEV), beta.to(DEV), 1e-6, y=y)
    torch.cuda.synchronize()
    assert bool((buf[:band] == -5.0).all()) and bool((buf[-band:] == -5.0).all())
    ref = blocks.layernorm_f64(parity.bf16_tensor_to_f64(x), gamma.numpy(), beta.numpy(), 1e-6)
    got = parity.bf16_tensor_to_f64(y)
    # fp32 statistics and one rounding to bf16
    assert np.all(np.abs(got - ref) <= 2.0 ** -8 * np.abs(ref) + 1e-3), float(np.abs(got - ref).max())
