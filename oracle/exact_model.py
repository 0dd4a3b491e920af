"""Exact-rational second model of the fold -- TEST INFRASTRUCTURE ONLY.

An independent restatement of the arithmetic the C oracle performs, written
with ``fractions.Fraction`` so that no hardware floating point is involved:
every bf16 pattern is decoded to an exact rational, every addition is carried
out exactly and then rounded to the binary32 grid (24-bit significand,
round to nearest, ties to even, gradual underflow, overflow to infinity), and
the final value is rounded to the bf16 grid (8-bit significand, same rules).
IEEE 754 fixes all of this; the collective's definition only fixes the order
(left fold over ranks 0..N-1, starting from rank 0's value).

It is slow (pure Python) and meant for brute force over small inputs.
"""
from __future__ import annotations

from fractions import Fraction
from typing import Sequence, Tuple

# A value is ("nan",), ("inf", sign) or ("fin", sign, Fraction magnitude); sign is 0 or 1.
Value = Tuple

_EMIN = -126
_EMAX = 127


def decode_bf16(h: int) -> Value:
    sign, expo, mant = (h >> 15) & 1, (h >> 7) & 0xFF, h & 0x7F
    if expo == 0xFF:
        return ("inf", sign) if mant == 0 else ("nan",)
    if expo == 0:
        return ("fin", sign, Fraction(mant, 1 << 7) * Fraction(1, 1 << 126))
    return ("fin", sign, (1 + Fraction(mant, 1 << 7)) * Fraction(2) ** (expo - 127))


def _floor_log2(x: Fraction) -> int:
    e = x.numerator.bit_length() - x.denominator.bit_length()
    if Fraction(2) ** e > x:
        e -= 1
    return e


def _round_mag(mag: Fraction, precision: int):
    """Round a positive rational to ``precision`` significant bits; None means overflow."""
    if mag == 0:
        return mag
    e = max(_floor_log2(mag), _EMIN)
    quantum = Fraction(2) ** (e - precision + 1)
    q = mag / quantum
    n = q.numerator // q.denominator
    rem = q - n
    if rem > Fraction(1, 2) or (rem == Fraction(1, 2) and n % 2 == 1):
        n += 1
    out = n * quantum
    if out >= Fraction(2) ** (_EMAX + 1):
        return None
    return out


def add_binary32(a: Value, b: Value) -> Value:
    """IEEE 754 binary32 addition, round to nearest even, of two values already on that grid."""
    if a[0] == "nan" or b[0] == "nan":
        return ("nan",)
    if a[0] == "inf" or b[0] == "inf":
        if a[0] == "inf" and b[0] == "inf":
            return a if a[1] == b[1] else ("nan",)
        return a if a[0] == "inf" else b
    sa = -a[2] if a[1] else a[2]
    sb = -b[2] if b[1] else b[2]
    s = sa + sb
    if s == 0:
        # exact zero sum: -0 only when both operands are negative (round-to-nearest rule)
        return ("fin", 1 if (a[1] and b[1]) else 0, Fraction(0))
    sign = 1 if s < 0 else 0
    mag = _round_mag(abs(s), 24)
    return ("inf", sign) if mag is None else ("fin", sign, mag)


def encode_bf16(v: Value) -> int:
    """Round a binary32-grid value to bf16 (nearest even) and return its bit pattern."""
    if v[0] == "nan":
        return 0x7FFF
    if v[0] == "inf":
        return (v[1] << 15) | 0x7F80
    sign = v[1]
    mag = _round_mag(v[2], 8)
    if mag is None:
        return (sign << 15) | 0x7F80
    if mag == 0:
        return sign << 15
    e = _floor_log2(mag)
    if e < _EMIN:                                   # subnormal: mag = m * 2^-133
        m = mag * (1 << 133)
        assert m.denominator == 1 and 0 < m.numerator < 128
        return (sign << 15) | int(m.numerator)
    frac = mag / Fraction(2) ** e - 1
    m = frac * 128
    assert m.denominator == 1 and 0 <= m.numerator < 128
    return (sign << 15) | ((e + 127) << 7) | int(m.numerator)


# ---- the same model for binary16 and binary32 storage ----------------------------------------------------

_FORMATS = {            # name: (exponent bits, fraction bits)
    "bf16": (8, 7), "f16": (5, 10), "f32": (8, 23),
}


def decode(h: int, fmt: str) -> Value:
    ebits, fbits = _FORMATS[fmt]
    bias = (1 << (ebits - 1)) - 1
    sign = (h >> (ebits + fbits)) & 1
    expo = (h >> fbits) & ((1 << ebits) - 1)
    mant = h & ((1 << fbits) - 1)
    if expo == (1 << ebits) - 1:
        return ("inf", sign) if mant == 0 else ("nan",)
    if expo == 0:
        return ("fin", sign, Fraction(mant, 1 << fbits) * Fraction(2) ** (1 - bias))
    return ("fin", sign, (1 + Fraction(mant, 1 << fbits)) * Fraction(2) ** (expo - bias))


def _round_mag_fmt(mag: Fraction, precision: int, emin: int, emax: int):
    if mag == 0:
        return mag
    e = max(_floor_log2(mag), emin)
    quantum = Fraction(2) ** (e - precision + 1)
    q = mag / quantum
    n = q.numerator // q.denominator
    rem = q - n
    if rem > Fraction(1, 2) or (rem == Fraction(1, 2) and n % 2 == 1):
        n += 1
    out = n * quantum
    return None if out >= Fraction(2) ** (emax + 1) else out


def encode(v: Value, fmt: str) -> int:
    ebits, fbits = _FORMATS[fmt]
    bias = (1 << (ebits - 1)) - 1
    top = ((1 << ebits) - 1) << fbits
    sbit = ebits + fbits
    if v[0] == "nan":
        return (1 << sbit) - 1                      # canonical: all ones below the sign bit
    if v[0] == "inf":
        return (v[1] << sbit) | top
    sign = v[1]
    mag = _round_mag_fmt(v[2], fbits + 1, 1 - bias, bias)
    if mag is None:
        return (sign << sbit) | top
    if mag == 0:
        return sign << sbit
    e = _floor_log2(mag)
    if e < 1 - bias:
        m = mag / Fraction(2) ** (1 - bias - fbits)
        assert m.denominator == 1
        return (sign << sbit) | int(m.numerator)
    m = (mag / Fraction(2) ** e - 1) * (1 << fbits)
    assert m.denominator == 1
    return (sign << sbit) | ((e + bias) << fbits) | int(m.numerator)


def fold_fmt(column: Sequence[int], fmt: str) -> int:
    """Left fold with binary32 partial sums over values stored in `fmt`, then one round to `fmt`."""
    acc = decode(int(column[0]), fmt)
    for h in column[1:]:
        acc = add_binary32(acc, decode(int(h), fmt))
    return encode(acc, fmt)


def is_nan_fmt(h: int, fmt: str) -> bool:
    ebits, fbits = _FORMATS[fmt]
    return ((h >> fbits) & ((1 << ebits) - 1)) == (1 << ebits) - 1 and (h & ((1 << fbits) - 1)) != 0


def fold(column: Sequence[int]) -> int:
    """Left fold in rank order with binary32 partial sums, then one round to bf16."""
    acc = decode_bf16(int(column[0]))
    for h in column[1:]:
        acc = add_binary32(acc, decode_bf16(int(h)))
    return encode_bf16(acc)


def is_nan_bf16(h: int) -> bool:
    return (h & 0x7F80) == 0x7F80 and (h & 0x007F) != 0
