"""Exact-rational statement of the NVFP4 quantizer -- TEST INFRASTRUCTURE.

Pure Python on ``fractions.Fraction``; no floating point hardware is involved, so
it is independent of the C oracle's arithmetic and of the CUDA path.  Used to pin
the C oracle on small inputs and on exhaustive scalar sweeps.

Two definitions of Q(x) = S * Pi_FP4(x / S) (paper Section 2) with S = s_block * T:

* ``quantize_block_rounded``  -- every intermediate (a/(6T), s*T, 1/d, x*rcp) is
  rounded to IEEE binary32 nearest-even, the operation order the C oracle and the
  CUDA kernel follow (the normative one: bit-exactness is defined on it);
* ``quantize_block_exact``    -- the same with real-number division: the nearest
  grid point of x / (s*T), ties to the even code.  Informative: it bounds how far
  the FP32 sequence is from the paper's formula (they differ only on values a
  rounded reciprocal nudges across a tie).
"""
from __future__ import annotations

from fractions import Fraction

# E2M1: 1 sign, 2 exponent, 1 mantissa bit; bias 1; exponent field 0 is subnormal.
E2M1_MAGNITUDES = [
    (Fraction(m, 2) if e == 0 else Fraction(2) ** (e - 1) * (1 + Fraction(m, 2)))
    for e in range(4) for m in range(2)
]

# E4M3 (fn): bias 7; exponent field 0 subnormal m * 2^-9; codes 0x00..0x7E finite.
E4M3_VALUES = [
    (Fraction(m, 512) if e == 0 else Fraction(2) ** (e - 7) * (1 + Fraction(m, 8)))
    for e in range(16) for m in range(8)
][:127]


def nearest_even_index(a: Fraction, grid) -> int:
    """Index of the grid value nearest to a >= 0; ties go to the even index; values
    above the last grid value saturate to it."""
    if a >= grid[-1]:
        return len(grid) - 1
    best, best_d = 0, abs(a - grid[0])
    for i in range(1, len(grid)):
        d = abs(a - grid[i])
        if d < best_d or (d == best_d and i % 2 == 0):
            best, best_d = i, d
    return best


def bf16_bits_to_fraction(h: int) -> Fraction:
    s, e, m = (h >> 15) & 1, (h >> 7) & 0xFF, h & 0x7F
    if e == 0xFF:
        raise ValueError("non-finite BF16")
    mag = Fraction(m, 128) * Fraction(2) ** -126 if e == 0 else (1 + Fraction(m, 128)) * Fraction(2) ** (e - 127)
    return -mag if s else mag


def round_f32(v: Fraction) -> Fraction:
    """IEEE binary32 round-to-nearest-even of a rational (finite range only)."""
    if v == 0:
        return v
    s, a = (-1 if v < 0 else 1), abs(v)
    # exponent e with 2^e <= a < 2^(e+1)
    e = a.numerator.bit_length() - a.denominator.bit_length()
    if Fraction(2) ** e > a:
        e -= 1
    if Fraction(2) ** (e + 1) <= a:
        e += 1
    e = max(e, -126)
    quantum = Fraction(2) ** (e - 23)
    n = a / quantum
    fl = n.numerator // n.denominator
    rem = n - fl
    if rem > Fraction(1, 2) or (rem == Fraction(1, 2) and fl % 2 == 1):
        fl += 1
    return s * fl * quantum


def e2m1_code(y: Fraction, negative: bool) -> int:
    return (8 if negative else 0) | nearest_even_index(abs(y), E2M1_MAGNITUDES)


def quantize_block_rounded(x_bits, T: Fraction):
    """Normative FP32 sequence on one block of 16 BF16 bit patterns -> (scale byte, 16 codes)."""
    xs = [bf16_bits_to_fraction(h) for h in x_bits]
    a = max(abs(x) for x in xs)
    c = round_f32(6 * T)
    v = round_f32(a / c)
    sb = nearest_even_index(v, E4M3_VALUES)
    if sb == 0:
        rcp = Fraction(0)
    else:
        d = round_f32(E4M3_VALUES[sb] * T)
        rcp = round_f32(1 / d)
    codes = [e2m1_code(round_f32(x * rcp), bool(h >> 15)) for x, h in zip(xs, x_bits)]
    return sb, codes


def quantize_block_exact(x_bits, T: Fraction):
    """Real-number division everywhere -> (scale byte, 16 codes)."""
    xs = [bf16_bits_to_fraction(h) for h in x_bits]
    a = max(abs(x) for x in xs)
    sb = nearest_even_index(a / (6 * T), E4M3_VALUES)
    if sb == 0:
        codes = [(8 if h >> 15 else 0) for h in x_bits]
    else:
        S = E4M3_VALUES[sb] * T
        codes = [e2m1_code(x / S, bool(h >> 15)) for x, h in zip(xs, x_bits)]
    return sb, codes


def dequantize_exact(sb: int, codes, T: Fraction):
    out = []
    for c in codes:
        mag = E2M1_MAGNITUDES[c & 7] * E4M3_VALUES[sb] * T
        out.append(-mag if c & 8 else mag)
    return out
