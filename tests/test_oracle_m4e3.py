"""Pins for the oracle's decode of the paper's own W/A byte format (Sec. 3.1, "M4E3 with flex-bias") and for the
chains that run on it.  No GPU.  The pins: hand-worked codes, products and chains (tests/golden/m4e3_input_format.txt),
the value set that Eq. 2 defines for (M, E, b) = (4, 3, 0), the exact-rational coding, and the arithmetic facts that
make this input format different from E4M3 (products of ten significant bits)."""
import os
from fractions import Fraction

import numpy as np

from oracle import lba_oracle as orc
from oracle import lba_exact as ex

M4E3 = 4          # flags bit2 of the product format
UF = 1


def _rows(path, kind):
    with open(path) as fh:
        for line in fh:
            parts = line.split()
            if parts and parts[0] == kind:
                yield parts[1:]


def test_hand_worked_codes_products_and_chains(golden_dir):
    path = os.path.join(golden_dir, "m4e3_input_format.txt")
    n = 0
    for code, want in _rows(path, "code"):
        assert orc.decode_m4e3(int(code, 16)) == float(want)
        assert ex.decode_m4e3(int(code, 16)) == Fraction(float(want))
        n += 1
    for xc, wc, M, E, b, rnd, want in _rows(path, "product"):
        prod = (int(M), int(E), int(b), int(rnd), UF | M4E3)
        wide = (23, 8, 127, int(rnd), UF)            # an accumulator that changes nothing: the result is Q_prod(x w)
        got = orc.dot(prod, wide, orc.SEQUENTIAL, 1, [int(xc, 16)], [int(wc, 16)])
        assert got == float(want), (xc, wc, got)
        assert ex.dot(prod, wide, 0, 1, [int(xc, 16)], [int(wc, 16)]) == Fraction(float(want))
        n += 1
    for xc, wc, K, bp, ba, rnd, want in _rows(path, "chain"):
        prod, acc = (7, 4, int(bp), int(rnd), UF | M4E3), (7, 4, int(ba), int(rnd), UF)
        xs, ws = [int(xc, 16)] * int(K), [int(wc, 16)] * int(K)
        assert orc.dot(prod, acc, orc.SEQUENTIAL, 1, xs, ws) == float(want)
        assert ex.dot(prod, acc, 0, 1, xs, ws) == Fraction(float(want))
        n += 1
    assert n == 21


def test_value_set_is_that_of_eq2_for_m4_e3_b0():
    # Eq. 2 with M = 4, E = 3, b = 0: magnitudes 2^e (1 + m/16), e = 0..7; the code e = m = 0 is zero instead of 2^0
    want = sorted({Fraction(2) ** e * (1 + Fraction(m, 16)) for e in range(8) for m in range(16)} - {Fraction(1)})
    pos = sorted(ex.decode_m4e3(c) for c in range(1, 128))
    assert pos == want and len(pos) == 127
    assert ex.decode_m4e3(0) == 0 and ex.decode_m4e3(0x80) == 0
    assert pos[-1] == ex.r_of(4, 3, 0) == 248                     # the largest code is R_OF of Eq. 2
    assert pos[0] == ex.r_uf(0) * Fraction(17, 16)                 # the smallest sits one step above R_UF = 2^-b
    for c in range(256):
        v = ex.decode_m4e3(c)
        assert ex.decode_m4e3(c ^ 0x80) == -v                      # sign bit
        assert Fraction(orc.decode_m4e3(c)) == v                   # the C++ decode agrees on every code
        for rnd in (0, 1):                                         # every value is a fixed point of Q_{4,3,0}
            assert ex.quantise((4, 3, 0, rnd, 1), v) == v
            assert orc.quantise((4, 3, 0, rnd, 1), float(v)) == float(v)
    mags = [ex.decode_m4e3(c) for c in range(128)]
    assert all(a < b for a, b in zip(mags, mags[1:]))              # monotone in the code


def test_products_have_up_to_ten_significant_bits_so_q_prod_cuts():
    # E4M3 x E4M3 products fit 8 significant bits and pass Q_prod with M = 7 untouched; here they do not
    widest, cut = 0, 0
    for a in range(1, 128):
        for b in range(a, 128):
            p = ex.decode_m4e3(a) * ex.decode_m4e3(b)
            n = p.numerator
            while n % 2 == 0:
                n //= 2
            widest = max(widest, n.bit_length())
            cut += ex.quantise((7, 4, 0, 0, 1), p) != p
    assert widest == 10 and cut > 1000
    assert ex.decode_m4e3(0x7F) ** 2 == 61504 < ex.r_of(7, 4, 0)   # the bias rule: b_prod = 0 holds every product
    assert ex.decode_m4e3(0x7F) ** 2 > ex.r_of(7, 4, 1)


def test_all_code_pairs_k1_cpp_against_rationals():
    codes = np.arange(256, dtype=np.uint8)
    A = np.repeat(codes, 256).reshape(-1, 1)
    B = codes.reshape(-1, 1)
    one = np.ones(1, dtype=np.float32)
    for prod, acc in (((7, 4, 0, 0, 5), (7, 4, -2, 0, 1)), ((7, 4, 0, 1, 5), (7, 4, -2, 1, 1)),
                      ((4, 3, -8, 0, 5), (4, 3, -10, 0, 1)), ((7, 4, 2, 0, 5), (7, 4, 0, 0, 1)), ((5, 5, 16, 1, 4), (5, 5, 14, 1, 0))):
        got = orc.gemm(A[::256][:, :], B, one, one, None, prod, acc, orc.SEQUENTIAL, 1)   # [256 x][256 w]
        for xi in range(0, 256, 1):
            x = ex.decode_m4e3(xi)
            for wi in range(0, 256, 5):
                want = ex.quantise(acc, ex.quantise(prod, x * ex.decode_m4e3(wi)))
                assert Fraction(float(got[xi, wi])) == want, (prod, acc, xi, wi)


def test_random_chains_cpp_against_rationals():
    rng = np.random.default_rng(20240114)
    for trial in range(40):
        K = int(rng.integers(1, 70))
        xs = rng.integers(0, 256, K).astype(np.uint8)
        ws = rng.integers(0, 256, K).astype(np.uint8)
        rnd = trial % 2
        prod, acc = (7, 4, 0, rnd, 5), (7, 4, -2, rnd, 1)
        for order, chunk in ((0, 1), (1, 16), (1, 5)):
            got = orc.dot(prod, acc, order, chunk, xs, ws)
            assert Fraction(got) == ex.dot(prod, acc, order, chunk, xs, ws)
