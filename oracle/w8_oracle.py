"""CPU oracle of the 8-bit weight encoding (test infrastructure; only tests and the benchmark's CPU leg import it).

Section 4 of the paper closes with a list of next steps whose second item is 8-bit quantisation of the weights;
it fixes no format.  The reading taken here: each matrix the projections stream is stored as e4m3 codes
(1 sign bit, 4 exponent bits with bias 7, 3 fraction bits; exponent field 0 holds the sub-normals
fraction/8 * 2^-6; the all-ones pattern 0x7f is not a number, so the largest magnitude is 0x7e = 448) with one
scale per output row, the scale being the smallest power of two s with max|w| <= 448 s (s = 1 for a row of zeros).
A weight w is encoded as the code whose value is nearest to w / s, a tie going to the code with the even bit
pattern, magnitudes beyond 448 to 448; it is decoded as value(code) * s.  Everything below is that definition
written out with a table of the 127 non-negative code values; no conversion routine of a library is used.

Pins (tests/test_oracle_pins.py): the table against the format's published landmarks, ties, the scale rule at its
boundaries, decode(encode(x)) = x on the code grid, the half-ulp error bound, and agreement with torch's own
float8_e4m3fn cast on in-range values.
"""
from __future__ import annotations

import numpy as np

E4M3_MAX = 448.0


def code_values() -> np.ndarray:
    """Value of each of the 256 bit patterns (float64; NaN for 0x7f and 0xff)."""
    v = np.empty(256, dtype=np.float64)
    for c in range(256):
        e, m = (c >> 3) & 15, c & 7
        if e == 15 and m == 7:
            mag = np.nan
        elif e == 0:
            mag = (m / 8.0) * 2.0 ** -6
        else:
            mag = (1.0 + m / 8.0) * 2.0 ** (e - 7)
        v[c] = -mag if c & 0x80 else mag
    return v


_VAL = code_values()
_POS = _VAL[:127]            # values of codes 0x00..0x7e, ascending


def encode(x) -> np.ndarray:
    """Nearest code of every entry of x (float64 array), ties to the even pattern, saturating at +-448."""
    x = np.asarray(x, dtype=np.float64)
    a = np.minimum(np.abs(x), E4M3_MAX)
    hi = np.searchsorted(_POS, a, side="left")            # first code with value >= a
    hi = np.minimum(hi, 126)
    lo = np.maximum(hi - 1, 0)
    d_lo, d_hi = a - _POS[lo], _POS[hi] - a
    pick_hi = (d_hi < d_lo) | ((d_hi == d_lo) & (hi % 2 == 0))
    code = np.where(pick_hi, hi, lo).astype(np.uint8)
    return np.where(np.signbit(x), code | np.uint8(0x80), code).astype(np.uint8)


def row_scales(w) -> np.ndarray:
    """Per row: the smallest power of two s with max|w| <= 448 s; 1 for a row of zeros."""
    amax = np.max(np.abs(np.asarray(w, dtype=np.float64)), axis=1)
    pos = amax > 0.0
    a = np.where(pos, amax, 1.0)
    e = np.ceil(np.log2(a / E4M3_MAX))
    e = np.where(a > E4M3_MAX * 2.0 ** e, e + 1, e)            # (guards the rounding of log2, either way)
    e = np.where(a <= E4M3_MAX * 2.0 ** (e - 1), e - 1, e)
    assert np.all(a <= E4M3_MAX * 2.0 ** e) and np.all(a > E4M3_MAX * 2.0 ** (e - 1))
    return np.where(pos, 2.0 ** e, 1.0).astype(np.float32)


def quantise_rows(w):
    """(codes uint8 [rows, cols], scales float32 [rows]) of a matrix [rows, cols]."""
    s = row_scales(w)
    return encode(np.asarray(w, dtype=np.float64) / s.astype(np.float64)[:, None]), s


def dequantise_rows(codes, scales) -> np.ndarray:
    return (_VAL[np.asarray(codes, dtype=np.uint8)] * np.asarray(scales, dtype=np.float64)[:, None]).astype(np.float32)


MATRICES = ("w_qkv", "w_o", "w_fc", "w_proj")


def model_on_the_grid(weights: dict) -> dict:
    """The model whose streamed matrices (the four per layer and the embedding / output-head table) are replaced by
    decode(encode(.)): every such entry is then a code value times a power of two, which both bf16 and the 8-bit
    format represent exactly.  Everything else is passed through."""
    out = dict(weights)
    for k in MATRICES:
        out[k] = [dequantise_rows(*quantise_rows(t)) for t in weights[k]]
    out["wte"] = dequantise_rows(*quantise_rows(weights["wte"]))
    return out
