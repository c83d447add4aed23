"""8-bit floating point (e4m3) for the oracle: decode table, quantiser, exact widening to bf16.

Test infrastructure only (never imported by the library).  The format is the published OCP 8-bit
floating-point "E4M3" (the tensor cores' e4m3 operand type): 1 sign bit, 4 exponent bits with bias 7, 3
mantissa bits; exponent field 0 holds the subnormals m/8 * 2^-6; there are no infinities, the one NaN
per sign is S.1111.111, so the largest finite magnitude is 1.75 * 2^8 = 448.

The masked convolution with 8-bit operands is still Eq. 4 / Eq. 6 of the paper on the values the codes
stand for: every e4m3 value is exactly a bf16 value (3 mantissa bits, exponents -9..8), so the codes are
widened exactly and handed to the same fp64 convolution oracle.
"""
from __future__ import annotations

import numpy as np

E4M3_MAX = 448.0


def e4m3_decode_table() -> np.ndarray:
    """float64 [256]: the value of every code, written out from the format's definition (NaN for the
    two NaN codes)."""
    out = np.empty(256, dtype=np.float64)
    for code in range(256):
        sign = -1.0 if code & 0x80 else 1.0
        e = (code >> 3) & 0xF
        m = code & 0x7
        if e == 0xF and m == 0x7:
            out[code] = np.nan
        elif e == 0:
            out[code] = sign * (m / 8.0) * 2.0 ** -6
        else:
            out[code] = sign * (1.0 + m / 8.0) * 2.0 ** (e - 7)
    return out


def e4m3_decode(codes: np.ndarray) -> np.ndarray:
    return e4m3_decode_table()[np.asarray(codes, dtype=np.uint8)]


def quantize_e4m3(x: np.ndarray) -> np.ndarray:
    """Nearest e4m3 value, ties to the code with an even mantissa, magnitudes beyond 448 saturate to
    448; the sign of the input is kept (so -0.0 and tiny negatives give the code of -0).  x: finite.
    Written as a search over the table, not as bit manipulation."""
    x = np.asarray(x, dtype=np.float64)
    table = e4m3_decode_table()
    pos_codes = np.arange(0x7F)                 # 0 .. 0x7E: the finite non-negative codes, ascending in value
    pos_vals = table[pos_codes]
    mag = np.minimum(np.abs(x), E4M3_MAX)
    hi = np.searchsorted(pos_vals, mag, side="left")          # first value >= mag
    hi = np.clip(hi, 0, len(pos_vals) - 1)
    lo = np.maximum(hi - 1, 0)
    d_lo = mag - pos_vals[lo]
    d_hi = pos_vals[hi] - mag
    take_hi = (d_hi < d_lo) | ((d_hi == d_lo) & ((pos_codes[hi] & 1) == 0))
    code = np.where(take_hi, pos_codes[hi], pos_codes[lo]).astype(np.uint8)
    return code | (np.signbit(x).astype(np.uint8) << 7)


def e4m3_to_bf16_bits(codes: np.ndarray) -> np.ndarray:
    """uint16 bf16 bit patterns of the same values (exact: every e4m3 value is a bf16 value)."""
    v = e4m3_decode(codes).astype(np.float32)
    bits = v.view(np.uint32)
    assert not (bits & 0xFFFF).any(), "an e4m3 value needed more than bf16's 8 significant bits"
    return (bits >> 16).astype(np.uint16)


def abs_code(codes: np.ndarray) -> np.ndarray:
    """Magnitude field of e4m3 codes as an integer that orders like |w| (+0 == -0)."""
    return (np.asarray(codes, dtype=np.uint8) & np.uint8(0x7F)).astype(np.int32)
