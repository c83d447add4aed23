"""Pins of the general N:M mask bookkeeping of the oracle (CPU only)."""
import itertools
import math

import numpy as np
import pytest

from oracle import masks

CASES = [(2, 4), (1, 4), (3, 4), (1, 2), (2, 8), (4, 8), (1, 8)]


@pytest.mark.parametrize("N,M", CASES)
def test_pattern_matrix_is_all_keep_N_of_M_vectors_in_lexicographic_order(N, M):
    D = masks.nm_pattern_matrix(N, M)
    assert D.shape == (M, math.comb(M, N))                       # n = C(M, N) (Sec. 3.1)
    assert (D.sum(axis=0) == N).all()
    cols = [tuple(D[:, p]) for p in range(D.shape[1])]
    assert len(set(cols)) == len(cols)
    # brute force: every 0/1 vector of length M with N ones appears
    brute = {v for v in itertools.product((0, 1), repeat=M) if sum(v) == N}
    assert set(cols) == brute
    kept = [tuple(i for i in range(M) if c[i]) for c in cols]
    assert kept == sorted(kept) == list(masks.nm_kept_positions(N, M))


def test_two_of_four_is_the_special_case_already_pinned():
    assert masks.nm_kept_positions(2, 4) == tuple(masks.KEPT_POSITIONS)
    assert np.array_equal(masks.nm_pattern_matrix(2, 4), masks.pattern_matrix())
    rng = np.random.default_rng(1)
    s = rng.normal(size=(500, 6)).astype(np.float32)
    assert np.array_equal(masks.nm_select_from_logits(s), masks.select_from_logits(s))
    bits = rng.integers(0, 2 ** 16, size=(500, 4)).astype(np.uint16)
    mags = (bits & 0x7FFF).astype(np.int64)
    assert np.array_equal(masks.nm_select_from_magnitude(mags, 2), masks.select_from_magnitude(bits))
    pat = rng.integers(0, 6, size=500).astype(np.uint8)
    assert np.array_equal(masks.nm_mask_from_pattern(pat, 2, 4, (500, 4)), masks.mask_from_pattern(pat, (500, 4)))


@pytest.mark.parametrize("N,M", CASES)
def test_magnitude_selection_is_the_best_pattern_by_enumeration(N, M):
    rng = np.random.default_rng(10 * N + M)
    mags = rng.integers(0, 5, size=(3000, M))          # a small alphabet: many ties
    got = masks.nm_select_from_magnitude(mags, N)
    pats = masks.nm_kept_positions(N, M)
    for g in range(mags.shape[0]):
        best = min(range(len(pats)), key=lambda p: (-int(mags[g, list(pats[p])].sum()), pats[p]))
        assert got[g] == best
        kept = list(pats[got[g]])
        dropped = [i for i in range(M) if i not in kept]
        if dropped:
            assert mags[g, kept].min() >= mags[g, dropped].max()


@pytest.mark.parametrize("N,M", CASES)
def test_mask_blocks_are_columns_of_D_and_keep_N(N, M):
    rng = np.random.default_rng(N + 100 * M)
    shape = (6, 3, 2 * M)
    G = 6 * 3 * 2
    pat = rng.integers(0, math.comb(M, N), size=G).astype(np.uint8)
    m = masks.nm_mask_from_pattern(pat, N, M, shape)
    blocks = m.reshape(-1, M)
    assert (blocks.sum(axis=1) == N).all()
    D = masks.nm_pattern_matrix(N, M)
    assert all(np.array_equal(blocks[g], D[:, pat[g]]) for g in range(G))
    # block g covers elements [M g, M g + M) of the flattened (row-major) weight
    assert np.array_equal(m.reshape(-1)[M * 5:M * 6], D[:, pat[5]])
