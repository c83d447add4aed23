"""Host-side logic of the library that needs no GPU: the folded descriptor's geometry, the planner's
folding rule, the pattern counts of N:M masks and the scratch size of the one-call input gradient."""
import math

import pytest

from paper_2411_00288_b200 import api


def _extent(n, k, s, p, d):
    return (n + 2 * p - d * (k - 1) - 1) // s + 1


@pytest.mark.parametrize("W,KW,s,p,d,f", [(56, 3, 1, 1, 1, 2), (56, 3, 1, 1, 1, 4), (57, 3, 2, 1, 1, 2), (30, 5, 1, 4, 2, 2),
                                          (112, 4, 1, 0, 1, 2), (24, 1, 2, 0, 1, 3), (16, 7, 2, 3, 1, 2)])
def test_folded_descriptor_covers_exactly_the_original_outputs(W, KW, s, p, d, f):
    Wo = _extent(W, KW, s, p, d)
    desc = api.make_desc(2, 9, W, 16, 24, 3, KW, stride=(1, s), pad=(1, p), dil=(1, d))
    if Wo % f:
        with pytest.raises(api.SsconvError):
            api.ssconv_fold_desc(desc, f)
        return
    fd = api.ssconv_fold_desc(desc, f)
    assert (fd.C_out, fd.KW, fd.stride_w, fd.dil_w, fd.pad_w) == (24 * f, (f - 1) * s + (KW - 1) * d + 1, f * s, 1, p)
    assert (fd.KH, fd.stride_h, fd.pad_h, fd.dil_h, fd.C_in, fd.H, fd.W, fd.N) == (3, 1, 1, 1, 16, 9, W, 2)
    # the folded layer's own output extent is the original's divided by f, and pixel f i + j of the original
    # reads, at tap kw, the column pixel i of the folded layer reads at tap j s + kw d
    assert _extent(W, fd.KW, fd.stride_w, p, 1) * f == Wo
    for i in range(Wo // f):
        for j in range(f):
            for kw in range(KW):
                assert (f * i + j) * s - p + kw * d == i * fd.stride_w - p + (j * s + kw * d)


def test_fold_factor_rule():
    assert api.ssconv_fold_factor(api.make_desc(1, 56, 56, 64, 64, 3, 3, 1, 1)) == 2
    assert api.ssconv_fold_factor(api.make_desc(1, 56, 56, 64, 32, 5, 5, 1, 2)) == 2
    assert api.ssconv_fold_factor(api.make_desc(1, 56, 56, 64, 64, 3, 3, 2, 1)) == 2      # (3 + 2) / 6 <= 0.85
    assert api.ssconv_fold_factor(api.make_desc(1, 56, 56, 64, 64, 1, 1, 1, 0)) == 1      # nothing shared between taps
    assert api.ssconv_fold_factor(api.make_desc(1, 56, 56, 64, 72, 3, 3, 1, 1)) == 1      # more than 64 output channels
    assert api.ssconv_fold_factor(api.make_desc(1, 56, 57, 64, 64, 3, 3, 1, 1)) == 1      # odd output width


@pytest.mark.parametrize("N,M", [(2, 4), (1, 4), (3, 4), (1, 2), (2, 8), (4, 8), (7, 8), (1, 1), (8, 8)])
def test_nm_pattern_count_is_the_binomial_coefficient(N, M):
    assert api.ssconv_nm_patterns(N, M) == math.comb(M, N)


def test_input_gradient_scratch_size():
    fwd = api.ssconv_sizes(api.make_desc(1, 8, 8, 64, 64, 1, 1)).ws_bytes_sparse     # the convolutions' own K-split scratch

    def r256(v):
        return (v + 255) // 256 * 256

    # unit stride: the reversed weights + the convolution's scratch
    d = api.make_desc(2, 14, 14, 64, 128, 3, 3, 1, 1)
    assert api.ssconv_dgrad_ws_bytes(d) == r256(64 * 9 * 128 * 2) + fwd
    # 3x3 stride 2: four classes in one convolution on a 2 x 2 window: weights [4 * 64, 2, 2, 128], tensor [2, 8, 8, 256]
    d = api.make_desc(2, 14, 14, 64, 128, 3, 3, 2, 1)
    assert api.ssconv_dgrad_ws_bytes(d) == r256(256 * 4 * 128 * 2) + r256(2 * 8 * 8 * 256 * 2) + fwd
    # 1x1 stride 2: one class with a tap, its own convolution: weights [64, 1, 1, 128], tensor [2, 7, 7, 64]
    d = api.make_desc(2, 14, 14, 64, 128, 1, 1, 2, 0)
    assert api.ssconv_dgrad_ws_bytes(d) == r256(64 * 128 * 2) + r256(2 * 7 * 7 * 64 * 2) + fwd
    # strided and dilated: the plain route: reversed weights [64, 3, 3, 64] + dy spread over all 9 x 9 filter
    # placements of unit stride (H + 2 pad - dil (K - 1) = 9) + the convolution's scratch
    d = api.make_desc(1, 9, 9, 64, 64, 3, 3, 2, 2, 2)
    assert api.ssconv_dgrad_ws_bytes(d) == r256(64 * 9 * 64 * 2) + r256(9 * 9 * 64 * 2) + fwd
    with pytest.raises(api.SsconvError):
        api.ssconv_dgrad_ws_bytes(api.make_desc(1, 8, 8, 64, 64, 1, 1, 1, 1))      # padding beyond the filter's reach
