"""CPU oracle for 2:4 mask selection, mask assembly and the logical compressed form.

TEST INFRASTRUCTURE, not a product path: only the tests, the smoke check and the
benchmark's CPU-baseline leg may import this module.  It shares no code with the CUDA
library and imports nothing from the package.

What it restates (all from Sec. 3.1 and Fig. 1 of the paper):

* N:M sparsity with N=2 zeros in every block of M=4 contiguous elements.  The paper's
  printed pattern count is garbled; the number of ways to keep 2 of 4 is C(4,2) = 6.
* The pattern matrix D (Eq. 2) holds one pattern per column, here 4 x 6, columns in
  lexicographic order of the kept positions: {0,1},{0,2},{0,3},{1,2},{1,3},{2,3}
  (the paper does not fix a column order; any order is a relabelling of the logits).
* Eq. 1: the hard choice is z = onehot(argmax_i [g_i + log pi_i]).  The scores handed to
  this oracle already contain whatever Gumbel noise the caller wants; ties go to the
  lowest index (the paper is silent on ties).
* Eq. 2: the mask is assembled row-major from blocks b = D z, one block per group.
* Fig. 1: the structured representation keeps only the two non-zeros of each block and a
  2-bit position index for each of them.

Group order: a weight tensor [C_out, KH, KW, C_in] is read as the row-major matrix
W in R^{C_out x (KH*KW*C_in)} of Eq. 5/6 with columns ordered (kh, kw, c_in); group g
covers the 4 consecutive input channels 4q..4q+3 at one (c_out, kh, kw).
"""
from __future__ import annotations

import numpy as np

# Kept positions of the six patterns, lexicographic.
KEPT_POSITIONS = ((0, 1), (0, 2), (0, 3), (1, 2), (1, 3), (2, 3))


def pattern_matrix() -> np.ndarray:
    """D of Eq. 2 as a 4 x 6 array of 0/1: column p is pattern p."""
    D = np.zeros((4, 6), dtype=np.uint8)
    for p, (a, b) in enumerate(KEPT_POSITIONS):
        D[a, p] = 1
        D[b, p] = 1
    return D


def select_from_logits(scores: np.ndarray) -> np.ndarray:
    """Eq. 1 without the one-hot: index of the largest of the 6 scores of each group.

    scores: float32 [G, 6].  A strict '>' scan from i = 0 keeps the first maximum.
    Comparisons are made on the float32 values as given (no arithmetic on them).
    """
    s = np.asarray(scores, dtype=np.float32)
    assert s.ndim == 2 and s.shape[1] == 6
    best = np.zeros(s.shape[0], dtype=np.uint8)
    best_val = s[:, 0].copy()
    for i in range(1, 6):
        better = s[:, i] > best_val
        best[better] = i
        best_val[better] = s[better, i]
    return best


def _abs_bits(w_bits: np.ndarray) -> np.ndarray:
    """Magnitude of bf16 bit patterns as an integer that orders like |w| (+0 == -0)."""
    return (np.asarray(w_bits, dtype=np.uint16) & np.uint16(0x7FFF)).astype(np.int32)


def select_from_magnitude(w_bits: np.ndarray, magnitudes: np.ndarray = None) -> np.ndarray:
    """Magnitude heuristic (Sec. 2, Sec. 3.2 closing remark): keep the two largest |w|.

    w_bits: uint16 bf16 bit patterns, any shape whose last axis is a multiple of 4 and
    whose flattening is the group order above.  Equal magnitudes: the lower position is
    kept first (a stable ordering), so the result is unique.  For weights of another type pass
    `magnitudes` (integers that order like |w|) instead; w_bits is then ignored.
    """
    a = (_abs_bits(w_bits) if magnitudes is None else np.asarray(magnitudes, dtype=np.int32)).reshape(-1, 4)
    # the plain definition: sort the four positions by decreasing magnitude with a stable sort (equal
    # magnitudes keep their order, so the lower position comes first) and keep the first two
    order = np.argsort(-a, axis=1, kind="stable")
    kept = np.sort(order[:, :2], axis=1)
    lut = {pos: p for p, pos in enumerate(KEPT_POSITIONS)}
    out = np.empty(a.shape[0], dtype=np.uint8)
    for (pa, pb), p in lut.items():
        out[(kept[:, 0] == pa) & (kept[:, 1] == pb)] = p
    return out


def mask_from_pattern(pattern: np.ndarray, shape) -> np.ndarray:
    """Eq. 2: mask of 0/1 bytes with the given weight shape from one pattern per group."""
    D = pattern_matrix()
    p = np.asarray(pattern, dtype=np.int64).reshape(-1)
    m = D[:, p].T  # [G, 4], block b = D z
    return np.ascontiguousarray(m.reshape(shape))


def apply_mask(w_bits: np.ndarray, mask: np.ndarray) -> np.ndarray:
    """Eq. 6's M .* W on bf16 bit patterns: dropped entries become +0, kept ones unchanged."""
    return np.where(mask.astype(bool), np.asarray(w_bits, dtype=np.uint16), np.uint16(0))


def logical_compress(w_bits: np.ndarray, pattern: np.ndarray):
    """Fig. 1's structured form, before any hardware tiling.

    Returns (values, codes): values uint16 [G, 2] = the two kept bf16 bit patterns in
    ascending position order; codes uint8 [G] = pos0 | pos1 << 2 (two 2-bit indices).
    """
    w = np.asarray(w_bits, dtype=np.uint16).reshape(-1, 4)
    p = np.asarray(pattern, dtype=np.int64).reshape(-1)
    pos = np.array(KEPT_POSITIONS, dtype=np.int64)[p]  # [G, 2]
    rows = np.arange(w.shape[0])
    values = np.stack([w[rows, pos[:, 0]], w[rows, pos[:, 1]]], axis=1)
    codes = (pos[:, 0] | (pos[:, 1] << 2)).astype(np.uint8)
    return values, codes


def logical_decompress(values: np.ndarray, codes: np.ndarray, shape) -> np.ndarray:
    """Inverse of logical_compress: scatter the kept values back, zeros elsewhere."""
    v = np.asarray(values, dtype=np.uint16).reshape(-1, 2)
    c = np.asarray(codes, dtype=np.int64).reshape(-1)
    out = np.zeros((v.shape[0], 4), dtype=np.uint16)
    rows = np.arange(v.shape[0])
    out[rows, c & 3] = v[:, 0]
    out[rows, (c >> 2) & 3] = v[:, 1]
    return out.reshape(shape)


# ---------------------------------------------------------------------------------------------------
# General N:M masks (Sec. 3.1: "N:M sparsity", blocks of M consecutive entries of a row of W of which
# N are kept, n = C(M, N) possible blocks as the columns of D).  The pattern order is lexicographic in
# the kept positions, which for 2:4 is the order of KEPT_POSITIONS above.
# ---------------------------------------------------------------------------------------------------
def nm_kept_positions(N: int, M: int):
    """The n = C(M, N) patterns as tuples of kept positions, lexicographic."""
    from itertools import combinations
    return tuple(combinations(range(M), N))


def nm_pattern_matrix(N: int, M: int) -> np.ndarray:
    """D in {0,1}^{M x n} of Eq. 2 for N:M blocks: column p has ones at the kept positions of pattern p."""
    pats = nm_kept_positions(N, M)
    D = np.zeros((M, len(pats)), dtype=np.uint8)
    for p, kept in enumerate(pats):
        D[list(kept), p] = 1
    return D


def nm_select_from_logits(scores: np.ndarray) -> np.ndarray:
    """Eq. 1 for any number of patterns: first maximum of each row of scores [G, n]."""
    s = np.asarray(scores, dtype=np.float32)
    best = np.zeros(s.shape[0], dtype=np.int64)
    best_val = s[:, 0].copy()
    for i in range(1, s.shape[1]):
        better = s[:, i] > best_val
        best[better] = i
        best_val[better] = s[better, i]
    return best.astype(np.uint8)


def nm_select_from_magnitude(magnitudes: np.ndarray, N: int) -> np.ndarray:
    """Keep the N largest of each block's M magnitudes (integers that order like |w|, [G, M]); equal
    magnitudes keep the lower position first: a stable sort by decreasing magnitude, first N kept."""
    a = np.asarray(magnitudes, dtype=np.int64)
    M = a.shape[1]
    order = np.argsort(-a, axis=1, kind="stable")
    kept = np.sort(order[:, :N], axis=1)
    lut = {pos: p for p, pos in enumerate(nm_kept_positions(N, M))}
    return np.array([lut[tuple(int(v) for v in row)] for row in kept], dtype=np.uint8)


def nm_mask_from_pattern(pattern: np.ndarray, N: int, M: int, shape) -> np.ndarray:
    """Eq. 2 for N:M blocks: 0/1 mask of the given weight shape, blocks of M along the last axis."""
    D = nm_pattern_matrix(N, M)
    blocks = D[:, np.asarray(pattern, dtype=np.int64)].T  # [G, M]
    return blocks.reshape(shape).astype(np.uint8)
