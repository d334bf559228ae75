"""Exact rational helpers for pinning fp32 arithmetic (pure Python, tiny inputs only).

Independent of the oracle: values are decoded from their bit patterns into Fractions and
rounded to binary32 with an explicit round-to-nearest-even, so a single-rounded fused
multiply-add can be checked without calling any fmaf."""
import struct
from fractions import Fraction


def f32_bits(x):
    return struct.unpack("<I", struct.pack("<f", x))[0]


def bits_f32(u):
    return struct.unpack("<f", struct.pack("<I", u & 0xFFFFFFFF))[0]


def frac_of_bits(u):
    """Exact value of a finite binary32 bit pattern."""
    sign = -1 if (u >> 31) else 1
    exp = (u >> 23) & 0xFF
    man = u & 0x7FFFFF
    assert exp != 0xFF, "finite values only"
    if exp == 0:
        return sign * Fraction(man, 1 << 149)
    return sign * Fraction((1 << 23) | man, 1) * Fraction(2) ** (exp - 150)


def round_to_f32_bits(fr):
    """Bit pattern of fr rounded to nearest-even binary32 (no overflow handling needed)."""
    if fr == 0:
        return 0
    sign = 0x80000000 if fr < 0 else 0
    m = abs(fr)
    e = m.numerator.bit_length() - m.denominator.bit_length()
    if Fraction(2) ** e > m:
        e -= 1
    assert Fraction(2) ** e <= m < Fraction(2) ** (e + 1)
    e = max(e, -126)
    quantum = Fraction(2) ** (e - 23)
    q = m / quantum
    n = q.numerator // q.denominator
    rem = q - n
    if rem > Fraction(1, 2) or (rem == Fraction(1, 2) and (n & 1)):
        n += 1
    val = n * quantum
    # re-encode: val = n * 2^(e-23), n <= 2^24
    if n == 0:
        return sign
    if n >= (1 << 24):
        n >>= 1
        e += 1
    if n < (1 << 23):                       # subnormal
        assert e == -126
        return sign | n
    return sign | ((e + 127) << 23) | (n & 0x7FFFFF)


def fma_f32_bits(alpha_bits, g_bits, e_bits):
    """Bits of round(alpha*g + e) with ONE rounding.  An exact zero result is +0 unless both
    addends are -0 (IEEE-754 round-to-nearest sign rule)."""
    p = frac_of_bits(alpha_bits) * frac_of_bits(g_bits)
    s = p + frac_of_bits(e_bits)
    if s == 0:
        p_neg = ((alpha_bits ^ g_bits) >> 31) & 1
        e_neg = (e_bits >> 31) & 1
        if p != 0 or frac_of_bits(e_bits) != 0:
            return 0                         # x + (-x) = +0
        return 0x80000000 if (p_neg and e_neg) else 0
    return round_to_f32_bits(s)
