"""Compressed cut-layer hand-off: 8-bit codes with one scale per token (arxiv 2407.00952).

TEST INFRASTRUCTURE ONLY.  Slow, obviously-correct checker for the CUDA codec; nothing in the
product path may import it and it shares no code or tables with the CUDA package.

The paper names the activations and activation gradients that cross the cut (Sec. III-B steps a2
and a4) as the communication cost of the method and, in Sec. V ("Efficiency in SplitLoRA"), names
quantisation as the direction for making that exchange cheaper; it fixes no format.  The format
stated here is this build's reading:

  * one row = one token's d features; scale[m] = absmax_m / 448, inv[m] = 448 / absmax_m
    (both fp32 divisions; a row of zeros has scale = inv = 0);
  * code[m, c] = E4M3(x[m, c] * inv[m]): the fp32 product rounded to the nearest value of the 8-bit
    floating-point format with 4 exponent and 3 mantissa bits (bias 7, subnormals, no infinities,
    largest finite value 448, the all-ones code reserved for NaN), ties to the even code,
    magnitudes above 448 clamped to 448;
  * the receiver restores x^[m, c] = value(code[m, c]) * scale[m] in fp32 and rounds once to the
    dtype of the hand-off buffer.

All decisions that produce an integer (the code) are taken in fp32, the precision the kernel uses.
The format itself is written out from its definition (sign, exponent, mantissa fields), not taken
from a library.

Parity status: pinned by tests/test_oracle_pins_handoff.py (the format's defining values, round
trip over all codes, ties, monotonicity, the half-step error bound, and torch's CPU conversion to
the same format as an independent routine).
"""
from __future__ import annotations

import numpy as np

F32 = np.float32
E4M3_MAX = 448.0
E4M3_NAN_CODE = 0x7F


def e4m3_value(code: int) -> float:
    """Value of one code, from the field definition: s eeee mmm, bias 7; e = 0 is subnormal
    (m / 8 * 2^-6); e = 15, m = 7 is NaN (there are no infinities)."""
    s, e, m = (code >> 7) & 1, (code >> 3) & 0xF, code & 7
    if e == 15 and m == 7:
        return float("nan")
    mag = (m / 8.0) * 2.0 ** -6 if e == 0 else (1.0 + m / 8.0) * 2.0 ** (e - 7)
    return -mag if s else mag


def e4m3_table() -> np.ndarray:
    """All 256 values, indexed by code (float64; every one is exact in fp32 as well)."""
    return np.array([e4m3_value(c) for c in range(256)], dtype=np.float64)


def e4m3_encode(y) -> np.ndarray:
    """Nearest code for each fp32 value: magnitude to the nearest of the 127 finite non-negative
    values (codes 0x00..0x7E in increasing order), halfway cases to the even code, above 448 to
    448; the sign bit is copied (so -0.0 and negative values that round to zero give 0x80)."""
    y = np.asarray(y, dtype=F32)
    mags = e4m3_table()[:E4M3_NAN_CODE]                  # increasing, 0 .. 448
    a = np.minimum(np.abs(y).astype(np.float64), E4M3_MAX)
    hi = np.clip(np.searchsorted(mags, a, side="left"), 0, len(mags) - 1)   # first value >= a
    lo = np.maximum(hi - 1, 0)
    d_hi, d_lo = mags[hi] - a, a - mags[lo]             # exact: operands are short binary fractions
    take_lo = (d_lo < d_hi) | ((d_lo == d_hi) & (lo % 2 == 0))
    code = np.where(take_lo, lo, hi).astype(np.uint8)
    return (code | (np.signbit(y).astype(np.uint8) << 7)).astype(np.uint8)


def quantize_rows(x):
    """x [M, d] (values of the hand-off dtype) -> (codes uint8 [M, d], scales fp32 [M])."""
    x = np.asarray(x, dtype=F32)
    absmax = np.max(np.abs(x), axis=1).astype(F32)
    nz = absmax > 0
    inv = np.zeros_like(absmax)
    scale = np.zeros_like(absmax)
    inv[nz] = F32(E4M3_MAX) / absmax[nz]
    scale[nz] = absmax[nz] / F32(E4M3_MAX)
    y = (x * inv[:, None]).astype(F32)                    # one fp32 product per element
    return e4m3_encode(y), scale


def round_to_bf16(v) -> np.ndarray:
    """fp32 -> nearest bf16 (ties to even), returned as fp32 values."""
    u = np.asarray(v, dtype=F32).view(np.uint32).astype(np.uint64)
    r = ((u + 0x7FFF + ((u >> 16) & 1)) >> 16) << 16
    return r.astype(np.uint32).view(F32)


def dequantize_rows(codes, scales, bf16: bool) -> np.ndarray:
    """(codes [M, d], scales [M]) -> x^ [M, d] as fp32 values (rounded to bf16 if the buffer is bf16)."""
    vals = e4m3_table().astype(F32)[np.asarray(codes, dtype=np.uint8)]
    out = (vals * np.asarray(scales, dtype=F32)[:, None]).astype(F32)
    return round_to_bf16(out) if bf16 else out


def handoff(x, bf16: bool) -> np.ndarray:
    """What the receiving side sees of x after the compressed hand-off."""
    codes, scales = quantize_rows(x)
    return dequantize_rows(codes, scales, bf16)
