"""GPU parity of the mask-learning step's kernels (soft mask, weight gradient, gradient to the
choice weights) against the fp64 oracle, on the same seeded inputs."""
import numpy as np
import pytest
import torch

from oracle import train as otrain
from oracle.conv import ConvShape, conv2d_f64
from paper_2411_00288_b200 import api, synth
from tests import parity

pytestmark = pytest.mark.gpu
DEV = "cuda:0"

# fp32 softmax against fp64: exp of an argument of magnitude a carries a relative error of about
# a * 2^-24; z <= 1
Z_ATOL, Z_RTOL = 1e-6, 3e-5
# one rounding to bf16 (8 significant bits: half an ulp is at most 2^-8 of the value) on top of fp32 arithmetic
WEFF_RTOL = 2.0 ** -8 * 1.01
# fp32 accumulation of exact products over up to 1e5 positions
WGRAD_REL_FRO, WGRAD_MAX_REL = 1e-4, 2e-4
LGRAD_REL_FRO = 1e-4


def _rel_fro(a, b):
    d = np.linalg.norm(b.reshape(-1))
    return float(np.linalg.norm((a - b).reshape(-1)) / d) if d > 0 else float(np.abs(a - b).max())


@pytest.mark.parametrize("G,tau,with_noise", [(1, 1.0, True), (255, 0.1, True), (4097, 0.5, False),
                                               (147456, 0.1, True), (589824, 2.0, True)])
def test_soft_mask_matches_oracle(G, tau, with_noise):
    g = torch.Generator().manual_seed(synth.SEED_BASE + 800 + G)
    logits = torch.randn((G, 6), generator=g)
    u = torch.rand((G, 6), generator=g, dtype=torch.float64).clamp_(1e-12, 1 - 1e-12)
    noise = (-torch.log(-torch.log(u))).float() if with_noise else None
    w = (torch.randn((G, 4), generator=g) * 0.05).to(torch.bfloat16)
    z, w_eff = api.ssconv_soft_mask(logits.to(DEV), None if noise is None else noise.to(DEV), tau, w.to(DEV))
    torch.cuda.synchronize()
    z_ref = otrain.soft_choice(logits.numpy(), None if noise is None else noise.numpy(), tau)
    zg = z.cpu().numpy().astype(np.float64)
    assert np.all(np.abs(zg - z_ref) <= Z_ATOL + Z_RTOL * z_ref), float(np.abs(zg - z_ref).max())
    we_ref = otrain.effective_weights(synth.bf16_bits(w), z_ref)
    we = parity.bf16_tensor_to_f64(w_eff)
    assert np.all(np.abs(we - we_ref) <= WEFF_RTOL * np.abs(we_ref) + 1e-30), float(np.abs(we - we_ref).max())


def test_soft_mask_outputs_are_optional_and_tau_is_checked():
    logits = torch.randn((64, 6)).to(DEV)
    w = torch.randn((64, 4)).to(torch.bfloat16).to(DEV)
    z, none = api.ssconv_soft_mask(logits, None, 0.3, w, want_w_eff=False)
    assert none is None and z.shape == (64, 6)
    none, w_eff = api.ssconv_soft_mask(logits, None, 0.3, w, want_z=False)
    assert none is None and w_eff.shape == w.shape
    with pytest.raises(api.SsconvError):
        api.ssconv_soft_mask(logits, None, 0.0, w)


@pytest.mark.parametrize("G,tau", [(3, 1.0), (1000, 0.1), (147456, 0.5)])
def test_mask_grad_matches_oracle(G, tau):
    g = torch.Generator().manual_seed(4242 + G)
    logits = torch.randn((G, 6), generator=g)
    w = (torch.randn((G, 4), generator=g) * 0.05).to(torch.bfloat16)
    up = torch.randn((G, 4), generator=g)
    z, _ = api.ssconv_soft_mask(logits.to(DEV), None, tau, w.to(DEV), want_w_eff=False)
    gl = api.ssconv_mask_grad(z, tau, w.to(DEV), up.to(DEV))
    torch.cuda.synchronize()
    # the kernel alone: same z on both sides
    ref_same_z = otrain.logit_grad(z.cpu().numpy(), tau, synth.bf16_bits(w), up.numpy())
    assert _rel_fro(gl.cpu().numpy().astype(np.float64), ref_same_z) <= 1e-5
    # the two kernels in sequence against the oracle's own z
    ref = otrain.logit_grad(otrain.soft_choice(logits.numpy(), None, tau), tau, synth.bf16_bits(w), up.numpy())
    assert _rel_fro(gl.cpu().numpy().astype(np.float64), ref) <= LGRAD_REL_FRO


WG_SWEEP = [
    # name                    N  H   W   Ci   Co  KH KW s  p  d
    ("pw_64",                 2, 9,  7,  64,  64, 1, 1, 1, 0, 1),
    ("pw_ragged_96to136",     3, 11, 5,  96, 136, 1, 1, 1, 0, 1),
    ("pw_s2",                 2, 10, 10, 64, 128, 1, 1, 2, 0, 1),
    ("c3_s1p1",               2, 12, 9,  64, 128, 3, 3, 1, 1, 1),
    ("c3_s2p1",               2, 13, 12, 128, 64, 3, 3, 2, 1, 1),
    ("c3_dil2",               1, 12, 12, 64,  64, 3, 3, 1, 2, 2),
    ("c5_p2_c32",             1, 9,  9,  32,  40, 5, 5, 1, 2, 1),
    ("c3_c8",                 2, 8,  8,  8,   8,  3, 3, 1, 1, 1),
    ("c3_7x7_maps",           9, 7,  7,  128, 256, 3, 3, 1, 1, 1),
    ("pw_deepK",              1, 6,  6,  1024, 64, 1, 1, 1, 0, 1),
    ("one_pixel",             1, 1,  1,  8,   8,  1, 1, 1, 0, 1),
    ("many_positions_split",  4, 40, 40, 64,  64, 3, 3, 1, 1, 1),
    ("pw_many_positions",     2, 64, 50, 64,  128, 1, 1, 1, 0, 1),
    # CTA-pair kernel: two tiles of 256 output channels (the second partly filled), a last group of k-blocks
    # with one, two and three members, a partial channel chunk, position ranges, one range only
    ("pair_two_n_tiles",      2, 9,  9,  64,  328, 3, 3, 1, 1, 1),
    ("pair_pw_5_kblocks",     2, 12, 10, 320, 200, 1, 1, 1, 0, 1),
    ("pair_pw_6_kblocks",     3, 9,  9,  384, 96,  1, 1, 1, 0, 1),
    ("pair_pw_3_kblocks",     2, 14, 14, 192, 768, 1, 1, 1, 0, 1),
    ("pair_c3_chunk_of_40",   2, 10, 11, 104, 72,  3, 3, 2, 1, 1),
    ("pair_split_ranges",     8, 28, 28, 256, 256, 3, 3, 1, 1, 1),
    ("pair_one_step",         1, 5,  5,  256, 256, 1, 1, 1, 0, 1),
]


def _check_wgrad(spec, seed=None):
    inp = synth.make_inputs(spec, seed=seed, x_only=True)
    tr = synth.make_train_inputs(spec, seed=seed)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    dw = api.ssconv_wgrad(api.desc_from_spec(spec), inp.x.to(DEV), tr.dy.to(DEV), dev_status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    ref = otrain.wgrad_f64(synth.bf16_bits(inp.x), synth.bf16_bits(tr.dy), spec.KH, spec.KW, spec.stride, spec.pad,
                           spec.dil)
    got = dw.cpu().numpy().astype(np.float64)
    assert got.shape == ref.shape
    return _rel_fro(got, ref), float(np.abs(got - ref).max() / max(np.abs(ref).max(), 1e-30))


@pytest.mark.parametrize("case", WG_SWEEP, ids=[c[0] for c in WG_SWEEP])
def test_wgrad_shape_sweep(case):
    name, N, H, W, Ci, Co, KH, KW, s, p, d = case
    spec = synth.LayerSpec(name, N, H, W, Ci, Co, KH, KW, s, p, d, config=8, index=WG_SWEEP.index(case))
    rel, mx = _check_wgrad(spec)
    assert rel <= WGRAD_REL_FRO and mx <= WGRAD_MAX_REL, f"{name}: rel_fro={rel:.3e} max_rel={mx:.3e}"


@pytest.mark.parametrize("index", [0, 1, 3, 4])
def test_wgrad_resnet18_layers_full_size(index):
    spec = [s for s in synth.config_layers(2) if not s.extra][index]
    rel, mx = _check_wgrad(spec)
    assert rel <= WGRAD_REL_FRO and mx <= WGRAD_MAX_REL, f"{spec.name}: rel_fro={rel:.3e} max_rel={mx:.3e}"


def test_wgrad_workspace_is_required_when_positions_are_split():
    spec = synth.config_layers(2)[0]
    desc = api.desc_from_spec(spec)
    assert api.ssconv_wgrad_ws_bytes(desc) > 0
    x = torch.zeros((spec.N, spec.H, spec.W, spec.C_in), dtype=torch.bfloat16, device=DEV)
    dy = torch.zeros((spec.N, spec.H_out, spec.W_out, spec.C_out), dtype=torch.bfloat16, device=DEV)
    tiny = torch.empty((16,), dtype=torch.uint8, device=DEV)
    with pytest.raises(api.SsconvError) as e:
        api.ssconv_wgrad(desc, x, dy, ws=tiny)
    assert e.value.status == 5


def test_one_mask_learning_step_of_a_layer():
    """soft mask -> dense forward with the effective weights -> weight gradient -> gradient of the
    choice weights, each stage against the oracle fed with the same bits."""
    spec = synth.LayerSpec("step", 4, 14, 14, 128, 128, 3, 3, 1, 1, 1, relu=False, has_bias=True, w_std="he",
                           config=8, index=60)
    tau = 0.5
    inp = synth.make_inputs(spec)
    tr = synth.make_train_inputs(spec)
    desc = api.desc_from_spec(spec)
    x, w = inp.x.to(DEV), inp.w.to(DEV)
    z, w_eff = api.ssconv_soft_mask(tr.logits.to(DEV), tr.noise.to(DEV), tau, w)
    y = api.ssconv_forward_dense(desc, x, w_eff, inp.bias.to(DEV))
    dw = api.ssconv_wgrad(desc, x, tr.dy.to(DEV))
    gl = api.ssconv_mask_grad(z, tau, w, dw)
    torch.cuda.synchronize()
    # forward: the oracle convolves with the effective weights the GPU rounded to bf16
    shp = ConvShape(spec.N, spec.H, spec.W, spec.C_in, spec.C_out, 3, 3, (1, 1), (1, 1), (1, 1), relu=False)
    y_ref = conv2d_f64(shp, synth.bf16_bits(inp.x), synth.bf16_bits(w_eff.cpu()), bias=inp.bias.numpy())
    rel, mx = parity.errors(parity.bf16_tensor_to_f64(y), y_ref)
    assert rel <= parity.REL_FRO_TOL and mx <= parity.MAX_ABS_TOL
    # backward: entirely from the oracle's own fp64 chain
    z_ref = otrain.soft_choice(tr.logits.numpy(), tr.noise.numpy(), tau)
    dw_ref = otrain.wgrad_f64(synth.bf16_bits(inp.x), synth.bf16_bits(tr.dy), 3, 3, 1, 1, 1)
    gl_ref = otrain.logit_grad(z_ref, tau, synth.bf16_bits(inp.w), dw_ref)
    assert _rel_fro(dw.cpu().numpy().astype(np.float64), dw_ref) <= WGRAD_REL_FRO
    assert _rel_fro(gl.cpu().numpy().astype(np.float64), gl_ref) <= LGRAD_REL_FRO


@pytest.mark.parametrize("n", [6, 6 * 1000 + 6, 6 * 147456])
def test_adamw_matches_oracle_over_several_steps(n):
    g = torch.Generator().manual_seed(999 + n)
    theta = torch.randn((n,), generator=g)
    m = torch.zeros(n)
    v = torch.zeros(n)
    th_d, m_d, v_d = theta.to(DEV), m.to(DEV), v.to(DEV)
    th_r, m_r, v_r = theta.numpy().astype(np.float64), np.zeros(n), np.zeros(n)
    # the call takes fp32 hyper-parameters: the oracle gets the values they round to
    lr, b1, b2, eps, wd = (float(np.float32(h)) for h in (1.0, 0.9, 0.999, 1e-8, 1e-4))
    for step in range(1, 5):
        grad = torch.randn((n,), generator=g) * (10.0 ** (step - 3))
        api.ssconv_adamw(th_d, grad.to(DEV), m_d, v_d, step, lr, b1, b2, eps, wd)
        th_r, m_r, v_r = otrain.adamw_step(th_r, grad.numpy(), m_r, v_r, step, lr, b1, b2, eps, wd)
    torch.cuda.synchronize()
    np.testing.assert_allclose(th_d.cpu().numpy(), th_r, rtol=2e-5, atol=2e-5)
    np.testing.assert_allclose(m_d.cpu().numpy(), m_r, rtol=1e-5, atol=1e-7)
    np.testing.assert_allclose(v_d.cpu().numpy(), v_r, rtol=1e-5, atol=1e-10)


def test_learning_the_mask_of_a_layer_reduces_its_distillation_loss():
    """Thirty steps of the whole loop on one layer, every kernel the library's own: the choice weights
    move so that the soft-masked layer reproduces the dense layer's output better, and the hard mask
    read off them afterwards beats the one read off the initial choice weights."""
    spec = synth.LayerSpec("learn", 2, 12, 12, 64, 64, 3, 3, 1, 1, 1, relu=False, has_bias=False, w_std="he",
                           config=8, index=70)
    inp = synth.make_inputs(spec)
    desc = api.desc_from_spec(spec)
    x, w = inp.x.to(DEV), inp.w.to(DEV)
    y_dense = api.ssconv_forward_dense(desc, x, w).float()
    g = torch.Generator().manual_seed(spec.seed + 1)
    logits = (torch.randn((spec.G, 6), generator=g) * 0.01).to(DEV)
    m, v = torch.zeros_like(logits), torch.zeros_like(logits)
    tau = 1.0

    def hard_loss(lg):
        pat = api.ssconv_select_mask(api.MASK_LOGITS_F32, lg, spec.G)
        wc, meta = api.ssconv_compress(desc, w, pat)
        return float(((api.ssconv_forward(desc, x, wc, meta).float() - y_dense) ** 2).mean())

    first_hard = hard_loss(logits)
    losses = []
    for step in range(1, 31):
        z, w_eff = api.ssconv_soft_mask(logits, None, tau, w)
        y = api.ssconv_forward_dense(desc, x, w_eff).float()
        diff = y - y_dense
        losses.append(float((diff ** 2).mean()))
        dy = (diff * (2.0 / diff.numel())).to(torch.bfloat16)  # the caller's loss gradient
        dw = api.ssconv_wgrad(desc, x, dy)
        gl = api.ssconv_mask_grad(z, tau, w, dw)
        api.ssconv_adamw(logits, gl, m, v, step, lr=0.3, weight_decay=1e-4)
    torch.cuda.synchronize()
    assert losses[-1] < 0.5 * losses[0], (losses[0], losses[-1])
    assert hard_loss(logits) < 0.8 * first_hard


DG_SWEEP = [
    # name          N  H   W   Ci   Co  KH KW p  d
    ("c3_p1",       2, 12, 9,  64,  128, 3, 3, 1, 1),
    ("pw",          2, 9,  7,  96,  136, 1, 1, 0, 1),
    ("c3_nopad",    1, 10, 10, 64,  64,  3, 3, 0, 1),
    ("c3_dil2",     1, 12, 12, 64,  64,  3, 3, 2, 2),
    ("c5_p2",       1, 9,  9,  32,  40,  5, 5, 2, 1),
    ("r18_128_28",  4, 28, 28, 128, 128, 3, 3, 1, 1),
]


@pytest.mark.parametrize("case", DG_SWEEP, ids=[c[0] for c in DG_SWEEP])
def test_input_gradient_through_the_dense_kernel_matches_oracle(case):
    name, N, H, W, Ci, Co, KH, KW, p, d = case
    spec = synth.LayerSpec(name, N, H, W, Ci, Co, KH, KW, 1, p, d, config=8, index=80 + DG_SWEEP.index(case))
    inp = synth.make_inputs(spec)
    g = torch.Generator().manual_seed(spec.seed + 5)
    dy = torch.randn((N, spec.H_out, spec.W_out, Co), generator=g).to(torch.bfloat16)
    desc = api.desc_from_spec(spec)
    desc_dx, w_t = api.ssconv_dgrad_prepare(desc, inp.w.to(DEV))
    assert (desc_dx.H, desc_dx.W, desc_dx.C_in, desc_dx.C_out) == (spec.H_out, spec.W_out, Co, Ci)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    dx = api.ssconv_forward_dense(desc_dx, dy.to(DEV), w_t, None, dev_status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0 and tuple(dx.shape) == (N, H, W, Ci)
    ref = otrain.dgrad_f64(synth.bf16_bits(dy), parity.bf16_tensor_to_f64(inp.w), H, W, 1, p, d)
    rel, mx = parity.errors(parity.bf16_tensor_to_f64(dx), ref)
    assert rel <= parity.REL_FRO_TOL and mx <= parity.MAX_ABS_TOL * max(1.0, float(np.abs(ref).max()) / 4.0), (rel, mx)


def test_input_gradient_is_refused_when_the_padding_exceeds_the_filters_reach():
    desc = api.make_desc(1, 8, 8, 64, 64, 1, 1, stride=1, pad=1)
    with pytest.raises(api.SsconvError) as e:
        api.ssconv_dgrad_prepare(desc, None)
    assert e.value.status == 3


# Strided layers: the gradient is first spread out with zeros.  H and W are chosen so that some
# sizes leave input rows and columns beyond the last filter placement (they must get zero gradient).
#              name            N  H   W   Ci   Co   KH KW s  p  d
DG_STRIDED = [
    ("s2_3x3",        2, 16, 16, 64,  64,  3, 3, 2, 1, 1),
    ("s2_3x3_odd",    2, 15, 18, 64,  96,  3, 3, 2, 1, 1),
    ("s2_1x1",        2, 14, 14, 128, 64,  1, 1, 2, 0, 1),
    ("s2_1x1_odd",    1, 13, 11, 64,  128, 1, 1, 2, 0, 1),
    ("s3_5x5",        1, 20, 17, 32,  40,  5, 5, 3, 2, 1),
    ("s2_3x3_dil2",   1, 18, 18, 64,  32,  3, 3, 2, 2, 2),
    ("s2_3x3_p0",     1, 12, 13, 32,  64,  3, 3, 2, 0, 1),
    ("r18_s2_64to128", 4, 56, 56, 64, 128, 3, 3, 2, 1, 1),
]


@pytest.mark.parametrize("case", DG_STRIDED, ids=[c[0] for c in DG_STRIDED])
def test_spread_gradient_is_bit_exact(case):
    name, N, H, W, Ci, Co, KH, KW, s, p, d = case
    spec = synth.LayerSpec(name, N, H, W, Ci, Co, KH, KW, s, p, d, config=8, index=90 + DG_STRIDED.index(case))
    g = torch.Generator().manual_seed(spec.seed + 5)
    dy = torch.randn((N, spec.H_out, spec.W_out, Co), generator=g).to(torch.bfloat16)
    desc = api.desc_from_spec(spec)
    got = api.ssconv_dgrad_spread(desc, dy.to(DEV)).cpu()
    Hz, Wz = H + 2 * p - d * (KH - 1), W + 2 * p - d * (KW - 1)
    ref = np.zeros((N, Hz, Wz, Co), dtype=np.uint16)
    ref[:, 0:s * (spec.H_out - 1) + 1:s, 0:s * (spec.W_out - 1) + 1:s, :] = synth.bf16_bits(dy)
    assert tuple(got.shape) == ref.shape
    np.testing.assert_array_equal(synth.bf16_bits(got), ref)


@pytest.mark.parametrize("case", DG_STRIDED, ids=[c[0] for c in DG_STRIDED])
def test_input_gradient_of_strided_layers_matches_oracle(case):
    name, N, H, W, Ci, Co, KH, KW, s, p, d = case
    spec = synth.LayerSpec(name, N, H, W, Ci, Co, KH, KW, s, p, d, config=8, index=90 + DG_STRIDED.index(case))
    inp = synth.make_inputs(spec)
    g = torch.Generator().manual_seed(spec.seed + 5)
    dy = torch.randn((N, spec.H_out, spec.W_out, Co), generator=g).to(torch.bfloat16)
    desc = api.desc_from_spec(spec)
    desc_dx, w_t = api.ssconv_dgrad_prepare(desc, inp.w.to(DEV))
    assert (desc_dx.stride_h, desc_dx.stride_w, desc_dx.C_in, desc_dx.C_out) == (1, 1, Co, Ci)
    dyz = api.ssconv_dgrad_spread(desc, dy.to(DEV))
    assert tuple(dyz.shape) == (N, desc_dx.H, desc_dx.W, Co)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    dx = api.ssconv_forward_dense(desc_dx, dyz, w_t, None, dev_status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0 and tuple(dx.shape) == (N, H, W, Ci)
    ref = otrain.dgrad_f64(synth.bf16_bits(dy), parity.bf16_tensor_to_f64(inp.w), H, W, s, p, d)
    rel, mx = parity.errors(parity.bf16_tensor_to_f64(dx), ref)
    assert rel <= parity.REL_FRO_TOL and mx <= parity.MAX_ABS_TOL * max(1.0, float(np.abs(ref).max()) / 4.0), (rel, mx)


# The one-call input gradient: unit stride through the reversed filter, strided layers through the residue
# classes of the input position (no zero-spread tensor).  Sentinel bands around dx.
#               name              N  H   W   Ci   Co   KH KW  s       p  d
DG_ONE_CALL = [
    ("s1_3x3",          2, 12, 9,  64,  128, 3, 3, (1, 1), 1, 1),
    ("s1_3x3_dil2",     1, 12, 12, 64,  64,  3, 3, (1, 1), 2, 2),
    ("s2_3x3",          2, 16, 16, 64,  64,  3, 3, (2, 2), 1, 1),
    ("s2_3x3_odd",      2, 15, 18, 64,  96,  3, 3, (2, 2), 1, 1),
    ("s2_1x1",          2, 14, 14, 128, 64,  1, 1, (2, 2), 0, 1),
    ("s2_1x1_odd",      1, 13, 11, 64,  128, 1, 1, (2, 2), 0, 1),
    ("s3_5x5",          1, 20, 17, 32,  40,  5, 5, (3, 3), 2, 1),
    ("s2_3x3_p0",       1, 12, 13, 32,  64,  3, 3, (2, 2), 0, 1),
    ("s2_3x3_p2",       1, 11, 12, 32,  32,  3, 3, (2, 2), 2, 1),
    ("s2_7x7_stem",     2, 30, 34, 8,   64,  7, 7, (2, 2), 3, 1),
    ("s4_4x4_patchify", 2, 16, 16, 8,   96,  4, 4, (4, 4), 0, 1),
    ("s2x1_3x3",        1, 14, 10, 64,  64,  3, 3, (2, 1), 1, 1),
    ("r18_s2_64to128",  4, 56, 56, 64,  128, 3, 3, (2, 2), 1, 1),
]


@pytest.mark.parametrize("case", DG_ONE_CALL, ids=[c[0] for c in DG_ONE_CALL])
def test_input_gradient_in_one_call_matches_oracle(case):
    name, N, H, W, Ci, Co, KH, KW, (sh, sw), p, d = case
    g = torch.Generator().manual_seed(synth.SEED_BASE + 4100 + DG_ONE_CALL.index(case))
    w = (torch.randn((Co, KH, KW, Ci), generator=g) * (2.0 / (KH * KW * Ci)) ** 0.5).to(torch.bfloat16)
    desc = api.make_desc(N, H, W, Ci, Co, KH, KW, stride=(sh, sw), pad=p, dil=d)
    Ho, Wo = api.ssconv_out_shape(desc)
    dy = torch.randn((N, Ho, Wo, Co), generator=g).to(torch.bfloat16)
    band = 4096
    buf = torch.full((N * H * W * Ci + 2 * band,), -7.0, dtype=torch.bfloat16, device=DEV)
    dx = buf[band:band + N * H * W * Ci].view(N, H, W, Ci)
    need = api.ssconv_dgrad_ws_bytes(desc)
    wsbuf = torch.full((need + 2 * band,), 0x5A, dtype=torch.uint8, device=DEV)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    api.ssconv_dgrad(desc, dy.to(DEV), w.to(DEV), dx=dx, ws=wsbuf[band:band + need], dev_status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    assert bool((buf[:band] == -7.0).all()) and bool((buf[-band:] == -7.0).all())
    assert bool((wsbuf[:band] == 0x5A).all()) and bool((wsbuf[-band:] == 0x5A).all())
    if sh == sw:
        ref = otrain.dgrad_f64(synth.bf16_bits(dy), parity.bf16_tensor_to_f64(w), H, W, sh, p, d)
    else:   # the oracle takes one stride: differentiate Eq. 4 term by term for the mixed case
        ref = np.zeros((N, H, W, Ci))
        dyf, wf = parity.bf16_tensor_to_f64(dy), parity.bf16_tensor_to_f64(w)
        for ho in range(Ho):
            for wo in range(Wo):
                for kh in range(KH):
                    for kw in range(KW):
                        h, ww = ho * sh - p + kh * d, wo * sw - p + kw * d
                        if 0 <= h < H and 0 <= ww < W:
                            ref[:, h, ww, :] += dyf[:, ho, wo, :] @ wf[:, kh, kw, :]
    rel, mx = parity.errors(parity.bf16_tensor_to_f64(dx), ref)
    assert rel <= parity.REL_FRO_TOL and mx <= parity.MAX_ABS_TOL * max(1.0, float(np.abs(ref).max()) / 4.0), (rel, mx)


def test_one_call_input_gradient_argument_rules():
    d = api.make_desc(1, 8, 8, 64, 64, 3, 3, stride=2, pad=1)
    dy = torch.zeros((1, 4, 4, 64), dtype=torch.bfloat16, device=DEV)
    w = torch.zeros((64, 3, 3, 64), dtype=torch.bfloat16, device=DEV)
    with pytest.raises(api.SsconvError) as e:
        api.ssconv_dgrad(d, dy, w, ws=torch.empty((16,), dtype=torch.uint8, device=DEV))
    assert e.value.status == 5          # workspace too small
    # strided and dilated: the plain route (spread gradient in the scratch), larger than the class route's
    assert api.ssconv_dgrad_ws_bytes(api.make_desc(1, 9, 9, 64, 64, 3, 3, stride=2, pad=2, dil=2)) > 9 * 9 * 64 * 2
    with pytest.raises(api.SsconvError) as e:
        api.ssconv_dgrad_ws_bytes(api.make_desc(1, 8, 8, 64, 64, 1, 1, stride=1, pad=1))
    assert e.value.status == 3          # padding beyond the filter's reach


@pytest.mark.parametrize("second", [(1, 1, 1, 0), (3, 3, 2, 1)], ids=["1x1", "3x3_stride2"])
def test_learning_the_masks_of_two_chained_layers(second):
    """Two layers trained together: the loss gradient reaches the first layer's choice weights through
    the second layer's input gradient (the one-call form and, on alternate steps, its parts with the
    gradient spread out first when that layer is strided).  Twenty-five steps
    must lower the loss."""
    KH2, KW2, st2, p2 = second
    s1 = synth.LayerSpec("chain1", 2, 12, 12, 64, 64, 3, 3, 1, 1, 1, relu=False, has_bias=False, w_std="he",
                         config=8, index=71)
    s2 = synth.LayerSpec("chain2", 2, 12, 12, 64, 128, KH2, KW2, st2, p2, 1, relu=False, has_bias=False, w_std="he",
                         config=8, index=72)
    i1, i2 = synth.make_inputs(s1), synth.make_inputs(s2)
    d1, d2 = api.desc_from_spec(s1), api.desc_from_spec(s2)
    x, w1, w2 = i1.x.to(DEV), i1.w.to(DEV), i2.w.to(DEV)
    target = api.ssconv_forward_dense(d2, api.ssconv_forward_dense(d1, x, w1), w2).float()
    g = torch.Generator().manual_seed(s1.seed + 9)
    l1 = (torch.randn((s1.G, 6), generator=g) * 0.01).to(DEV)
    l2 = (torch.randn((s2.G, 6), generator=g) * 0.01).to(DEV)
    m1, v1, m2, v2 = (torch.zeros_like(t) for t in (l1, l1, l2, l2))
    tau, losses = 1.0, []
    for step in range(1, 26):
        z1, e1 = api.ssconv_soft_mask(l1, None, tau, w1)
        z2, e2 = api.ssconv_soft_mask(l2, None, tau, w2)
        h = api.ssconv_forward_dense(d1, x, e1)
        y = api.ssconv_forward_dense(d2, h, e2).float()
        diff = y - target
        losses.append(float((diff ** 2).mean()))
        dy = (diff * (2.0 / diff.numel()) * 1e4).to(torch.bfloat16)  # scaled so that bf16 keeps it; Adam is scale-free
        g2 = api.ssconv_mask_grad(z2, tau, w2, api.ssconv_wgrad(d2, h, dy))
        if step % 2:   # both routes to the second layer's input gradient take turns
            dh = api.ssconv_dgrad(d2, dy, e2)
        else:
            dd, wt = api.ssconv_dgrad_prepare(d2, e2)
            dh = api.ssconv_forward_dense(dd, api.ssconv_dgrad_spread(d2, dy) if st2 > 1 else dy, wt, None)
        g1 = api.ssconv_mask_grad(z1, tau, w1, api.ssconv_wgrad(d1, x, dh))
        api.ssconv_adamw(l1, g1, m1, v1, step, lr=0.3)
        api.ssconv_adamw(l2, g2, m2, v2, step, lr=0.3)
    torch.cuda.synchronize()
    assert losses[-1] < 0.6 * losses[0], (losses[0], losses[-1])
