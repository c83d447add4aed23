"""Pins for the mask-selection / mask-assembly / compression oracle (CPU only)."""
import itertools
import os

import numpy as np
import pytest

from oracle import masks
from tests.brute import bf16_to_f64, f32_to_bf16_bits

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "patterns_2of4.txt")


def _golden_patterns():
    rows = []
    with open(GOLDEN) as f:
        for line in f:
            if line.startswith("#") or not line.strip():
                continue
            t = [int(v) for v in line.split()]
            rows.append(t)
    return rows


def test_pattern_matrix_matches_golden_and_is_exactly_all_2_of_4():
    D = masks.pattern_matrix()
    assert D.shape == (4, 6)
    rows = _golden_patterns()
    assert [r[0] for r in rows] == list(range(6))
    for p, *bits in rows:
        assert list(D[:, p]) == bits
    # every column keeps exactly 2 of 4 and the six columns are all distinct, hence they
    # are all C(4,2) = 6 legal patterns
    assert (D.sum(axis=0) == 2).all()
    assert len({tuple(D[:, p]) for p in range(6)}) == 6
    brute = sorted(c for c in itertools.product((0, 1), repeat=4) if sum(c) == 2)
    assert sorted(tuple(int(v) for v in D[:, p]) for p in range(6)) == brute


def test_select_logits_exhaustive_small_alphabet_first_max():
    # all 3^6 score vectors over {-1,0,1}: result is the first position of the maximum
    vecs = np.array(list(itertools.product((-1.0, 0.0, 1.0), repeat=6)), dtype=np.float32)
    got = masks.select_from_logits(vecs)
    for v, p in zip(vecs, got):
        mx = max(v)
        assert p == [i for i in range(6) if v[i] == mx][0]


def test_select_logits_matches_python_loop_and_softmax_argmax():
    rng = np.random.default_rng(7)
    s = rng.normal(size=(4096, 6)).astype(np.float32)
    got = masks.select_from_logits(s)
    # brute force in pure Python
    for g in range(0, 4096, 17):
        best, bv = 0, float(s[g, 0])
        for i in range(1, 6):
            if float(s[g, i]) > bv:
                best, bv = i, float(s[g, i])
        assert got[g] == best
    # Eq. 3 vs Eq. 1: softmax((.)/tau) is monotone, so its argmax is Eq. 1's argmax
    s64 = s.astype(np.float64)
    srt = np.sort(s64, axis=1)
    clear = (srt[:, -1] - srt[:, -2]) > 1e-3
    for tau in (0.1, 1.0):
        z = np.exp((s64 - s64.max(axis=1, keepdims=True)) / tau)
        z /= z.sum(axis=1, keepdims=True)
        assert (np.argmax(z, axis=1)[clear] == got[clear]).all()
    # adding the same constant to all six scores of a group does not move the argmax
    assert (masks.select_from_logits(s + np.float32(8.0)) == got).mean() > 0.999


def test_select_logits_onehot_picks_that_pattern():
    for p in range(6):
        s = np.full((3, 6), -2.0, dtype=np.float32)
        s[:, p] = 5.0
        assert (masks.select_from_logits(s) == p).all()


def _alphabet_bits():
    vals = np.array([0.0, -0.0, 0.5, -0.5, 1.0, -1.0, 1.5, 3.0], dtype=np.float32)
    return f32_to_bf16_bits(vals)


def _best_pattern_by_enumeration(mags):
    """Brute force over the six patterns, no sorting: the pattern whose kept pair has the largest
    magnitude sum (exact: the magnitudes are small dyadic numbers); among equal sums the one whose kept
    positions come first in lexicographic order, which is what "the lower position wins a tie" means."""
    best, best_key = None, None
    for p, (i, j) in enumerate(masks.KEPT_POSITIONS):
        key = (-(mags[i] + mags[j]), i, j)
        if best_key is None or key < best_key:
            best, best_key = p, key
    return best


def test_select_magnitude_exhaustive_vs_enumeration():
    alpha = _alphabet_bits()
    groups = np.array(list(itertools.product(alpha, repeat=4)), dtype=np.uint16)
    got = masks.select_from_magnitude(groups)
    mags = np.abs(bf16_to_f64(groups))
    D = masks.pattern_matrix()
    for g in range(groups.shape[0]):
        assert got[g] == _best_pattern_by_enumeration(mags[g])
        # the kept pair holds the two largest magnitudes: nothing dropped exceeds anything kept
        kept = list(masks.KEPT_POSITIONS[got[g]])
        dropped = [i for i in range(4) if i not in kept]
        assert min(mags[g, kept]) >= max(mags[g, dropped])
        # optimality: no other pattern keeps a larger magnitude sum (exact in fp64)
        sums = mags[g] @ D
        assert sums[got[g]] >= sums.max()


def test_select_magnitude_signs_and_zero_signs_do_not_matter():
    rng = np.random.default_rng(3)
    w = f32_to_bf16_bits(rng.normal(size=(2048, 4)).astype(np.float32))
    flipped = w ^ np.uint16(0x8000)
    assert (masks.select_from_magnitude(w) == masks.select_from_magnitude(flipped)).all()


def test_mask_from_pattern_blocks_are_columns_of_D_row_major():
    rng = np.random.default_rng(11)
    shape = (5, 3, 2, 8)  # C_out, KH, KW, C_in
    G = np.prod(shape) // 4
    pat = rng.integers(0, 6, size=G).astype(np.uint8)
    m = masks.mask_from_pattern(pat, shape)
    assert m.shape == shape and m.dtype == np.uint8
    blocks = m.reshape(-1, 4)
    assert (blocks.sum(axis=1) == 2).all()          # exactly 2 kept per group
    D = masks.pattern_matrix()
    legal = {tuple(D[:, p]) for p in range(6)}
    assert all(tuple(b) in legal for b in blocks)
    # group index is row-major over (c_out, kh, kw, c_in/4): spot-check one group by hand
    co, kh, kw, q = 3, 2, 1, 1
    g = ((co * 3 + kh) * 2 + kw) * 2 + q
    assert tuple(m[co, kh, kw, 4 * q:4 * q + 4]) == tuple(D[:, pat[g]])


def test_apply_mask_keeps_bits_and_matches_additive_perturbation_identity():
    rng = np.random.default_rng(5)
    shape = (4, 1, 1, 16)
    w = f32_to_bf16_bits(rng.normal(size=shape).astype(np.float32))
    pat = rng.integers(0, 6, size=16).astype(np.uint8)
    m = masks.mask_from_pattern(pat, shape)
    wm = masks.apply_mask(w, m)
    assert (wm[m == 1] == w[m == 1]).all()
    assert (wm[m == 0] == 0).all()
    # masking as an additive perturbation dW = (B - 1) .* W (proof of Lemma 3.3): W + dW = B .* W,
    # and ||dW||_inf <= ||W||_inf for the induced (row-sum) norm
    W = bf16_to_f64(w).reshape(4, 16)
    B = m.reshape(4, 16).astype(np.float64)
    dW = (B - 1.0) * W
    assert np.array_equal(W + dW, bf16_to_f64(wm).reshape(4, 16))
    assert np.abs(dW).sum(axis=1).max() <= np.abs(W).sum(axis=1).max()


def test_logical_compress_roundtrip_sizes_and_codes():
    rng = np.random.default_rng(9)
    shape = (8, 3, 3, 32)
    w = f32_to_bf16_bits(rng.normal(size=shape).astype(np.float32))
    w[0, 0, 0, :4] = 0  # a group of zeros is legal: the mask is positional
    pat = rng.integers(0, 6, size=np.prod(shape) // 4).astype(np.uint8)
    vals, codes = masks.logical_compress(w, pat)
    assert vals.shape == (pat.size, 2) and codes.shape == (pat.size,)
    # half the values plus 4 bits per group: 9/16 of the dense bytes ("roughly half", Fig. 1)
    dense_bytes = 2 * w.size
    assert vals.nbytes + codes.size // 2 == dense_bytes * 9 // 16
    # codes are two ascending 2-bit positions
    assert set(np.unique(codes)) <= {0x4, 0x8, 0xC, 0x9, 0xD, 0xE}
    for p, (a, b) in enumerate(masks.KEPT_POSITIONS):
        assert (codes[pat == p] == (a | (b << 2))).all()
    back = masks.logical_decompress(vals, codes, shape)
    assert np.array_equal(back, masks.apply_mask(w, masks.mask_from_pattern(pat, shape)))


@pytest.mark.parametrize("plant", ["swap_positions", "wrong_tiebreak"])
def test_pins_catch_planted_mistakes(plant, monkeypatch):
    """A pin that cannot fail pins nothing: plant a mistake in the oracle and see it caught."""
    if plant == "swap_positions":
        bad = list(masks.KEPT_POSITIONS)
        bad[1], bad[2] = bad[2], bad[1]
        monkeypatch.setattr(masks, "KEPT_POSITIONS", tuple(bad))
        D = masks.pattern_matrix()
        rows = _golden_patterns()
        assert any(list(D[:, p]) != bits for p, *bits in rows)
    else:
        # plant a tie-break that prefers the LATER position (an unstable sort would do this): the
        # exhaustive enumeration pin must notice on the groups that hold equal magnitudes
        def later_wins(w_bits):
            a = masks._abs_bits(w_bits).reshape(-1, 4)
            order = np.argsort(-a[:, ::-1], axis=1, kind="stable")   # ties -> higher position first
            kept = np.sort(3 - order[:, :2], axis=1)
            out = np.empty(a.shape[0], dtype=np.uint8)
            for p, (pa, pb) in enumerate(masks.KEPT_POSITIONS):
                out[(kept[:, 0] == pa) & (kept[:, 1] == pb)] = p
            return out
        monkeypatch.setattr(masks, "select_from_magnitude", later_wins)
        alpha = _alphabet_bits()
        groups = np.array(list(itertools.product(alpha, repeat=4)), dtype=np.uint16)
        got = masks.select_from_magnitude(groups)
        mags = np.abs(bf16_to_f64(groups))
        wrong = [g for g in range(groups.shape[0]) if got[g] != _best_pattern_by_enumeration(mags[g])]
        assert wrong, "the planted tie-break went unnoticed"
        # and only tie groups are affected: where all four magnitudes differ both rules agree
        assert all(len(set(mags[g])) < 4 for g in wrong)
