"""Eq. 2 and Eq. 4 of the paper in exact rational arithmetic.  TEST INFRASTRUCTURE ONLY.

Pure Python ``fractions.Fraction``: slow, for small cases.  It is written from the
formulas as printed (e, m, R_OF, R_UF, the three cases), not from the C++ oracle, and the
two are compared in the tests.  A format is ``(M, E, b, rounding, flags)``.
"""
from fractions import Fraction
import math


def decode_e4m3(code: int) -> Fraction:
    """Value of an OCP E4M3 byte: sign, 4 exponent bits (bias 7), 3 mantissa bits."""
    s, e, f = code >> 7, (code >> 3) & 15, code & 7
    if e == 15 and f == 7:
        raise ValueError("E4M3 NaN code")
    if e == 0:
        v = Fraction(f, 8) * Fraction(1, 2 ** 6)
    else:
        v = (1 + Fraction(f, 8)) * Fraction(2) ** (e - 7)
    return -v if s else v


def decode_m4e3(code: int) -> Fraction:
    """Value of a byte of the paper's W/A format (Sec. 3.1): sign, 3 exponent bits, 4 mantissa bits; Eq. 2 with
    (M, E, b) = (4, 3, 0) gives (-1)^s 2^e (1 + m/16); the code e = m = 0 is read as zero."""
    s, e, m = code >> 7, (code >> 4) & 7, code & 15
    if e == 0 and m == 0:
        return Fraction(0)
    v = (1 + Fraction(m, 16)) * Fraction(2) ** e
    return -v if s else v


def decoder(prod_fmt):
    """The byte decoder the product format names (flags bit2: M4E3 codes)."""
    return decode_m4e3 if (prod_fmt[4] & 4) else decode_e4m3


def r_of(M, E, b) -> Fraction:
    return Fraction(2) ** (2 ** E - b - 1) * (2 - Fraction(1, 2 ** M))


def r_uf(b) -> Fraction:
    return Fraction(2) ** (-b)


def _floor_log2(a: Fraction) -> int:
    # a > 0 ; exact: compare integers, never floats
    e = a.numerator.bit_length() - a.denominator.bit_length()
    if Fraction(2) ** e > a:
        e -= 1
    elif Fraction(2) ** (e + 1) <= a:
        e += 1
    assert Fraction(2) ** e <= a < Fraction(2) ** (e + 1)
    return e


def _round(v: Fraction, nearest: bool) -> int:
    fl = math.floor(v)
    if not nearest:
        return fl
    rem = v - fl
    if rem > Fraction(1, 2) or (rem == Fraction(1, 2) and fl % 2 == 1):
        return fl + 1
    return fl


def fixed_range(B, b):
    """(R_min, R_max) of Eq. 1."""
    return -Fraction(2) ** (B - b - 1), Fraction(2) ** (-b) * (2 ** (B - 1) - 1)


def quantise_fixed(fmt, x) -> Fraction:
    """Q^FIXED_{B,b}(x), Eq. 1, cases in the printed order, Round = floor; fmt = (B, 0, b, 0, flags) and flags bit1
    asks for two's-complement wrap-around (modulo 2^B) instead of the two saturating cases."""
    B, E, b, rounding, flags = fmt
    assert E == 0 and rounding == 0
    x = Fraction(x)
    lo, hi = fixed_range(B, b)
    if flags & 2:
        n = math.floor(x * Fraction(2) ** b)
        n = (n + 2 ** (B - 1)) % 2 ** B - 2 ** (B - 1)
        return Fraction(n) / Fraction(2) ** b
    if x <= lo:
        return lo
    if x >= hi:
        return hi
    return Fraction(math.floor(x * Fraction(2) ** b)) / Fraction(2) ** b


def quantise(fmt, x) -> Fraction:
    """Q^FLOAT_{M,E,b}(x), Eq. 2, cases in the printed order; zero is +0.  E = 0 selects Eq. 1."""
    M, E, b, rounding, flags = fmt
    if E == 0:
        return quantise_fixed(fmt, x)
    x = Fraction(x)
    if x == 0:
        return Fraction(0)
    sign = -1 if x < 0 else 1
    a = abs(x)
    top = r_of(M, E, b)
    if a >= top:
        return sign * top
    if (flags & 1) and a < r_uf(b):
        return Fraction(0)
    e = _floor_log2(a)
    m = Fraction(_round(Fraction(2) ** M * (a / Fraction(2) ** e - 1), rounding == 1), 2 ** M)
    y = Fraction(2) ** e * (m + 1)
    return sign * min(y, top)


def fmaq(prod_fmt, acc_fmt, x: Fraction, w: Fraction, s: Fraction) -> Fraction:
    """Eq. 4."""
    return quantise(acc_fmt, quantise(prod_fmt, x * w) + s)


def dot(prod_fmt, acc_fmt, order, chunk, xcodes, wcodes) -> Fraction:
    """Eq. 8-9 (order 0) or two-hierarchy chunked accumulation (order 1) over byte codes."""
    dec = decoder(prod_fmt)
    xs = [dec(int(c)) for c in xcodes]
    ws = [dec(int(c)) for c in wcodes]
    if order == 0:
        s = Fraction(0)
        for x, w in zip(xs, ws):
            s = fmaq(prod_fmt, acc_fmt, x, w, s)
        return s
    total = Fraction(0)
    for j in range(0, len(xs), chunk):
        c = Fraction(0)
        for x, w in zip(xs[j:j + chunk], ws[j:j + chunk]):
            c = fmaq(prod_fmt, acc_fmt, x, w, c)
        total = quantise(acc_fmt, c + total)
    return total


def last_overflow(prod_fmt, acc_fmt, xcodes, wcodes) -> int:
    """Sequential order: index of the last step with |Q_prod(x w) + S| >= R_OF(acc) (where the overflow
    straight-through estimator of App. D is 0), or -1."""
    M, E, b, _, _ = acc_fmt
    top = r_of(M, E, b)
    s = Fraction(0)
    last = -1
    for i, (xc, wc) in enumerate(zip(xcodes, wcodes)):
        t = quantise(prod_fmt, decode_e4m3(int(xc)) * decode_e4m3(int(wc))) + s
        if abs(t) >= top:
            last = i
        s = quantise(acc_fmt, t)
    return last


def ste_bits(prod_fmt, acc_fmt, order, chunk, xcodes, wcodes, kind, eps1=0.0, eps2=0.0):
    """STE value of every FMAq step (App. D), as two lists of 0/1: the steps of the first hierarchy and, in
    chunked order (order = 1), the folds of the chunk sums.  kind "OF": 1 iff |term + S| < R_OF(acc).
    kind "DIFF": 1 iff |z - S| > eps2 * (|u| + eps1), u the unquantised product (the chunk sum at a fold), every
    operation (the subtraction, the addition, the multiplication) rounded to binary32."""
    import numpy as np
    M, E, b, _, _ = acc_fmt
    top = r_of(M, E, b)

    def ste(term, u, s):
        z = quantise(acc_fmt, term + s)
        if kind == "OF":
            return z, int(abs(term + s) < top)
        den = np.float32(np.float32(float(abs(u))) + np.float32(eps1))
        thr = np.float32(np.float32(eps2) * den)
        d = np.float32(float(z)) - np.float32(float(s))      # z and S are binary32 numbers; one rounded subtraction
        return z, int(abs(d) > thr)

    first, second = [], []
    s = t = Fraction(0)
    n_in = 0
    for xc, wc in zip(xcodes, wcodes):
        xw = decode_e4m3(int(xc)) * decode_e4m3(int(wc))
        s, bit = ste(quantise(prod_fmt, xw), xw, s)
        first.append(bit)
        n_in += 1
        if order == 1 and n_in == chunk:
            t, bit = ste(s, s, t)
            second.append(bit)
            s, n_in = Fraction(0), 0
    if order == 1 and n_in > 0:
        t, bit = ste(s, s, t)
        second.append(bit)
    return first, second
