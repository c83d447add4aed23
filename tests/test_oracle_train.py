"""Pins for the mask-learning oracle (CPU only): soft choice (Eq. 3), soft block (Eq. 2),
effective weights (Eq. 6), the gradient to the choice weights, and the weight gradient of
the convolution.

Each function is fixed to something other than itself: defining ratios and closed forms,
the hard mask as the limit of small temperatures, central finite differences of the
(pinned) forward functions, the adjoint identity against the (pinned) convolution oracle,
and a nested-loop differentiation of Eq. 4 on tiny shapes.
"""
import numpy as np
import pytest

from oracle import masks, train
from oracle.conv import ConvShape, conv2d_f64
from tests.brute import bf16_to_f64, f32_to_bf16_bits


def _bits(rng, shape, scale=1.0):
    return f32_to_bf16_bits((rng.normal(size=shape) * scale).astype(np.float32))


def _gumbel(rng, shape):
    u = rng.uniform(1e-9, 1.0 - 1e-9, size=shape)
    return -np.log(-np.log(u))


# ---------------------------------------------------------------- Eq. 3
def test_soft_choice_is_a_distribution_with_the_defining_ratios():
    rng = np.random.default_rng(1)
    l = rng.normal(size=(50, 6)).astype(np.float32)
    g = _gumbel(rng, (50, 6)).astype(np.float32)
    for tau in (0.1, 0.5, 1.0, 3.0):
        z = train.soft_choice(l, g, tau)
        assert z.shape == (50, 6) and np.all(z > 0)
        np.testing.assert_allclose(z.sum(axis=1), 1.0, rtol=0, atol=1e-14)
        s = (l.astype(np.float64) + g.astype(np.float64)) / tau
        # z_i / z_j = exp(s_i - s_j): Eq. 3 without its normaliser
        for i, j in ((0, 5), (2, 3), (4, 1)):
            np.testing.assert_allclose(np.log(z[:, i]) - np.log(z[:, j]), s[:, i] - s[:, j], rtol=1e-9, atol=1e-9)


def test_soft_choice_closed_forms_and_invariances():
    z = train.soft_choice(np.full((3, 6), 0.7, np.float32), None, 0.3)
    np.testing.assert_allclose(z, 1.0 / 6.0, rtol=1e-15)
    rng = np.random.default_rng(2)
    l = rng.normal(size=(20, 6)).astype(np.float32)
    shift = rng.normal(size=(20, 1)).astype(np.float32)
    np.testing.assert_allclose(train.soft_choice(l.astype(np.float64) + shift, None, 0.5),
                               train.soft_choice(l, None, 0.5), rtol=1e-12)
    # two-point case: logits (a, 0, -inf...) approximated by very negative others
    l2 = np.full((1, 6), -1e4, np.float32)
    l2[0, 0], l2[0, 1] = 0.3, -0.2
    z2 = train.soft_choice(l2, None, 0.25)
    assert z2[0, 0] == pytest.approx(1.0 / (1.0 + np.exp((-0.2 - 0.3) / 0.25)), rel=1e-6)


def test_small_temperature_limit_is_the_hard_choice_of_eq1():
    rng = np.random.default_rng(3)
    l = rng.normal(size=(200, 6)).astype(np.float32)
    g = _gumbel(rng, (200, 6)).astype(np.float32)
    hard = masks.select_from_logits((l + g).astype(np.float32))
    z = train.soft_choice(l + g, None, 1e-4)
    assert np.array_equal(np.argmax(z, axis=1), hard)
    np.testing.assert_allclose(z[np.arange(200), hard], 1.0, atol=1e-9)
    b = train.soft_block(z)
    np.testing.assert_allclose(b, masks.mask_from_pattern(hard, (200, 4)).astype(np.float64), atol=1e-9)


# ---------------------------------------------------------------- Eq. 2 / Eq. 6 with soft z
def test_soft_block_sums_to_two_and_uniform_choice_gives_one_half():
    rng = np.random.default_rng(4)
    z = train.soft_choice(rng.normal(size=(64, 6)), None, 0.7)
    b = train.soft_block(z)
    np.testing.assert_allclose(b.sum(axis=1), 2.0, rtol=1e-13)
    assert np.all(b >= 0) and np.all(b <= 1 + 1e-15)
    # each position is kept by three of the six patterns
    np.testing.assert_allclose(train.soft_block(np.full((1, 6), 1 / 6)), 0.5, rtol=1e-15)
    # position 0 is kept by patterns 0, 1, 2; position 3 by patterns 2, 4, 5
    z1 = np.array([[0.1, 0.2, 0.3, 0.05, 0.15, 0.2]])
    b1 = train.soft_block(z1)[0]
    assert b1[0] == pytest.approx(0.6) and b1[3] == pytest.approx(0.65)
    assert b1[1] == pytest.approx(0.1 + 0.05 + 0.15) and b1[2] == pytest.approx(0.2 + 0.05 + 0.2)


def test_effective_weights_reduce_to_the_hard_mask_for_one_hot_choices():
    rng = np.random.default_rng(5)
    w = _bits(rng, (6, 3, 3, 8))
    pat = rng.integers(0, 6, size=w.size // 4)
    z = np.zeros((pat.size, 6))
    z[np.arange(pat.size), pat] = 1.0
    hard = masks.apply_mask(w, masks.mask_from_pattern(pat, w.shape))
    np.testing.assert_array_equal(train.effective_weights(w, z), bf16_to_f64(hard))
    # and scale elementwise otherwise
    z = train.soft_choice(rng.normal(size=(pat.size, 6)), None, 1.0)
    we = train.effective_weights(w, z).reshape(-1, 4)
    np.testing.assert_allclose(we, train.soft_block(z) * bf16_to_f64(w).reshape(-1, 4), rtol=0, atol=0)
    assert np.all(np.abs(we) <= np.abs(bf16_to_f64(w).reshape(-1, 4)))


# ---------------------------------------------------------------- gradient to the choice weights
@pytest.mark.parametrize("tau", [0.2, 1.0])
def test_logit_grad_matches_central_differences_of_the_forward(tau):
    rng = np.random.default_rng(6)
    G = 12
    l = rng.normal(size=(G, 6))
    g = _gumbel(rng, (G, 6))
    w = _bits(rng, (G, 4))
    up = rng.normal(size=(G, 4))  # dL/dW_eff of the linear loss L = sum(up * W_eff)

    def loss(lv):
        return float((up * train.effective_weights(w, train.soft_choice(lv, g, tau))).sum())

    z = train.soft_choice(l, g, tau)
    ana = train.logit_grad(z, tau, w, up)
    num = np.zeros_like(l)
    h = 1e-6
    for a in range(G):
        for i in range(6):
            lp, lm = l.copy(), l.copy()
            lp[a, i] += h
            lm[a, i] -= h
            num[a, i] = (loss(lp) - loss(lm)) / (2 * h)
    np.testing.assert_allclose(ana, num, rtol=2e-6, atol=2e-8)
    # a common shift of a group's logits changes nothing: the gradient sums to zero per group
    np.testing.assert_allclose(ana.sum(axis=1), 0.0, atol=1e-12)


def test_logit_grad_vanishes_for_saturated_choices():
    w = _bits(np.random.default_rng(7), (5, 4))
    l = np.full((5, 6), -200.0)
    l[:, 2] = 200.0
    z = train.soft_choice(l, None, 1.0)
    np.testing.assert_allclose(train.logit_grad(z, 1.0, w, np.ones((5, 4))), 0.0, atol=1e-30)


# ---------------------------------------------------------------- weight gradient of the convolution
WG_CASES = [
    # N  H  W  C  Co KH KW  s  p  d
    (1, 5, 5, 4, 3, 3, 3, 1, 1, 1),
    (2, 6, 7, 8, 5, 3, 3, 2, 1, 1),
    (1, 7, 6, 4, 2, 3, 3, 1, 2, 2),
    (2, 4, 6, 8, 4, 1, 1, 1, 0, 1),
    (1, 8, 8, 4, 4, 1, 1, 2, 0, 1),
    (1, 9, 7, 4, 2, 3, 3, 2, 0, 1),
]


def _loops_wgrad(x, dy, KH, KW, s, p, d):
    """Differentiate Eq. 4 term by term: every product x * w that enters y[n, ho, wo, co]
    hands dy[n, ho, wo, co] * x to that w."""
    N, H, W, C = x.shape
    _, Ho, Wo, Co = dy.shape
    dw = np.zeros((Co, KH, KW, C))
    for n in range(N):
        for ho in range(Ho):
            for wo in range(Wo):
                for kh in range(KH):
                    for kw in range(KW):
                        hi, wi = ho * s - p + kh * d, wo * s - p + kw * d
                        if 0 <= hi < H and 0 <= wi < W:
                            dw[:, kh, kw, :] += np.outer(dy[n, ho, wo, :], x[n, hi, wi, :])
    return dw


@pytest.mark.parametrize("case", WG_CASES)
def test_wgrad_matches_term_by_term_differentiation(case):
    N, H, W, C, Co, KH, KW, s, p, d = case
    rng = np.random.default_rng(hash(case) % (2 ** 32))
    x = _bits(rng, (N, H, W, C))
    Ho, Wo = train.conv_out_extent(H, KH, s, p, d), train.conv_out_extent(W, KW, s, p, d)
    dy = _bits(rng, (N, Ho, Wo, Co))
    got = train.wgrad_f64(x, dy, KH, KW, s, p, d)
    ref = _loops_wgrad(bf16_to_f64(x), bf16_to_f64(dy), KH, KW, s, p, d)
    np.testing.assert_allclose(got, ref, rtol=1e-12, atol=1e-12)


@pytest.mark.parametrize("case", WG_CASES)
def test_wgrad_is_the_adjoint_of_the_convolution_oracle(case):
    """<dy, conv(x, E)> = <wgrad(x, dy), E> for any E: the convolution is linear in its weights."""
    N, H, W, C, Co, KH, KW, s, p, d = case
    rng = np.random.default_rng(hash(case) % (2 ** 32) + 1)
    x = _bits(rng, (N, H, W, C))
    Ho, Wo = train.conv_out_extent(H, KH, s, p, d), train.conv_out_extent(W, KW, s, p, d)
    dy = _bits(rng, (N, Ho, Wo, Co))
    E = _bits(rng, (Co, KH, KW, C))
    y = conv2d_f64(ConvShape(N, H, W, C, Co, KH, KW, (s, s), (p, p), (d, d), relu=False), x, E)
    lhs = float((bf16_to_f64(dy) * y).sum())
    rhs = float((train.wgrad_f64(x, dy, KH, KW, s, p, d) * bf16_to_f64(E)).sum())
    assert lhs == pytest.approx(rhs, rel=1e-11, abs=1e-11)


def test_wgrad_of_an_impulse_gradient_is_the_input_patch():
    rng = np.random.default_rng(9)
    x = _bits(rng, (1, 6, 6, 4))
    dy = np.zeros((1, 6, 6, 3), dtype=np.uint16)
    dy[0, 0, 2, 1] = 0x3F80  # 1.0 at output pixel (0, 2), channel 1
    dw = train.wgrad_f64(x, dy, 3, 3, 1, 1, 1)
    assert np.all(dw[0] == 0) and np.all(dw[2] == 0)
    xf = bf16_to_f64(x)
    np.testing.assert_array_equal(dw[1, 0], 0.0)               # input row -1: padding
    np.testing.assert_array_equal(dw[1, 1], xf[0, 0, 1:4, :])   # kh = 1 -> input row 0, columns 1..3
    np.testing.assert_array_equal(dw[1, 2], xf[0, 1, 1:4, :])


def test_wgrad_of_a_1x1_filter_is_a_plain_matrix_product():
    rng = np.random.default_rng(10)
    x = _bits(rng, (2, 5, 4, 8))
    dy = _bits(rng, (2, 5, 4, 6))
    dw = train.wgrad_f64(x, dy, 1, 1, 1, 0, 1)
    ref = bf16_to_f64(dy).reshape(-1, 6).T @ bf16_to_f64(x).reshape(-1, 8)
    np.testing.assert_allclose(dw.reshape(6, 8), ref, rtol=1e-13)


# ---------------------------------------------------------------- gradient with respect to the input
@pytest.mark.parametrize("case", WG_CASES)
def test_dgrad_is_the_adjoint_of_the_convolution_oracle_in_x(case):
    """<dy, conv(e, w)> = <dgrad(dy, w), e> for any input e: the convolution is linear in its input."""
    N, H, W, C, Co, KH, KW, s, p, d = case
    rng = np.random.default_rng(hash(case) % (2 ** 32) + 2)
    Ho, Wo = train.conv_out_extent(H, KH, s, p, d), train.conv_out_extent(W, KW, s, p, d)
    dy = _bits(rng, (N, Ho, Wo, Co))
    w = _bits(rng, (Co, KH, KW, C))
    e = _bits(rng, (N, H, W, C))
    y = conv2d_f64(ConvShape(N, H, W, C, Co, KH, KW, (s, s), (p, p), (d, d), relu=False), e, w)
    lhs = float((bf16_to_f64(dy) * y).sum())
    dx = train.dgrad_f64(dy, bf16_to_f64(w), H, W, s, p, d)
    assert dx.shape == (N, H, W, C)
    assert lhs == pytest.approx(float((dx * bf16_to_f64(e)).sum()), rel=1e-11, abs=1e-11)


def test_dgrad_of_an_impulse_gradient_is_the_filter_placed_at_that_pixel():
    rng = np.random.default_rng(12)
    w = _bits(rng, (3, 3, 3, 4))
    dy = np.zeros((1, 5, 5, 3), dtype=np.uint16)
    dy[0, 2, 3, 1] = 0x3F80  # 1.0 at output pixel (2, 3), channel 1
    dx = train.dgrad_f64(dy, bf16_to_f64(w), 5, 5, 1, 1, 1)
    wf = bf16_to_f64(w)
    # output pixel (2, 3) read input pixels (1..3, 2..4) through taps (0..2, 0..2) of filter 1
    np.testing.assert_array_equal(dx[0, 1:4, 2:5, :], wf[1])
    dx[0, 1:4, 2:5, :] = 0
    assert not dx.any()


# ---------------------------------------------------------------- optimiser of the choice weights
def test_adamw_step_matches_the_library_optimiser_over_several_steps():
    import torch
    rng = np.random.default_rng(11)
    theta0 = rng.normal(size=(40, 6))
    grads = [rng.normal(size=(40, 6)) * (0.1 + 0.3 * i) for i in range(5)]
    lr, b1, b2, eps, wd = 0.05, 0.9, 0.999, 1e-8, 1e-2
    t = torch.tensor(theta0, dtype=torch.float64, requires_grad=True)
    opt = torch.optim.AdamW([t], lr=lr, betas=(b1, b2), eps=eps, weight_decay=wd)
    theta, m, v = theta0, np.zeros_like(theta0), np.zeros_like(theta0)
    for i, g in enumerate(grads, start=1):
        t.grad = torch.tensor(g, dtype=torch.float64)
        opt.step()
        theta, m, v = train.adamw_step(theta, g, m, v, i, lr, b1, b2, eps, wd)
        np.testing.assert_allclose(theta, t.detach().numpy(), rtol=1e-10, atol=1e-12)


def test_adamw_first_step_is_a_signed_unit_step_without_decay():
    g = np.array([3.0, -0.2, 1e-3])
    theta, m, v = train.adamw_step(np.zeros(3), g, np.zeros(3), np.zeros(3), 1, 0.5, 0.9, 0.999, 0.0, 0.0)
    np.testing.assert_allclose(theta, -0.5 * np.sign(g), rtol=1e-12)
    np.testing.assert_allclose(m, 0.1 * g, rtol=1e-12)
    np.testing.assert_allclose(v, 0.001 * g * g, rtol=1e-9)
