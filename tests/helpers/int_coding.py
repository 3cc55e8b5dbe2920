"""Eq. 2 and Eq. 4 once more, in 64-bit integer fixed point (numpy int64).  TEST HELPER.

A third coding of the quantiser, independent of the C++ oracle (exact dyadic carrier) and of the exact-rational
module: every value is an integer count of 2^-U, U large enough that every product, every quantised value and every
sum the tests form is an integer, and small enough that nothing leaves 63 bits.  Q is done with shifts, masks and
comparisons on whole arrays, so all code pairs times many running sums take seconds.  E4M3 values are multiples of
2^-9, products of 2^-18.
"""
import numpy as np


def e4m3_int(code, unit_exp):
    """Value of an E4M3 byte as an integer count of 2^-unit_exp (unit_exp >= 9)."""
    s, e, f = code >> 7, (code >> 3) & 15, code & 7
    assert not (e == 15 and f == 7)
    mag = f << (unit_exp - 9) if e == 0 else (8 + f) << (unit_exp - 10 + e) if unit_exp - 10 + e >= 0 else None
    assert mag is not None
    return -mag if s else mag


def quantise_int(v, M, E, b, rounding, flags, U):
    """Q^FLOAT_{M,E,b} of Eq. 2 on an int64 array of counts of 2^-U; returns counts of 2^-U."""
    v = np.asarray(v, dtype=np.int64)
    a = np.abs(v)
    emax = (1 << E) - b - 1
    # R_OF = (2^(M+1) - 1) * 2^(emax - M), R_UF = 2^-b, both in units of 2^-U
    assert emax - M + U >= 0 and emax + 1 + U < 62
    r_of = ((1 << (M + 1)) - 1) << (emax - M + U)
    r_uf = 1 << (U - b) if U >= b else 0             # below one unit: no non-zero count is under it
    # floor(log2 a) by bit length: 63 - leading zeros, via a float-free loop over the few possible positions
    e = np.zeros_like(a)
    t = a.copy()
    for sh in (32, 16, 8, 4, 2, 1):
        big = t >= (np.int64(1) << sh)
        e = np.where(big, e + sh, e)
        t = np.where(big, t >> sh, t)
    drop = np.maximum(e - M, 0)                      # low bits below the kept grid
    q = a >> drop
    rem = a - (q << drop)
    if rounding == 1:
        half = np.where(drop > 0, np.int64(1) << np.maximum(drop - 1, 0), np.int64(0))
        up = (drop > 0) & ((rem > half) | ((rem == half) & ((q & 1) == 1)))
        q = q + up.astype(np.int64)
    y = np.minimum(q << drop, r_of)                  # a carry past the top is brought back to R_OF
    y = np.where(a >= r_of, r_of, y)
    if flags & 1:
        y = np.where(a < r_uf, 0, y)
    y = np.where(a == 0, 0, y)
    return np.where(v < 0, -y, y)


def fmaq_int(prod, acc, x, w, s, U):
    """Eq. 4 on integer counts: x, w counts of 2^-(U/2) each (so that x*w is a count of 2^-U), s a count of 2^-U."""
    p = quantise_int(np.asarray(x, np.int64) * np.asarray(w, np.int64), *prod, U)
    return quantise_int(p + s, *acc, U)
