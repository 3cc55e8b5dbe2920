"""Pins for the oracle's scalar quantiser Q^FLOAT_{M,E,b} (Eq. 2 of the paper).

Nothing here uses a GPU.  The pins are: closed forms of Eq. 2 and textbook format maxima,
hand-worked values, invariants the definition implies (Table 1 error bounds, monotone,
odd, idempotent), IEEE conversions done by numpy / PyTorch (library routines), and an
independent exact-rational coding of the same formula.
"""
import os
from fractions import Fraction

import numpy as np
import pytest
import torch

from oracle import lba_oracle as orc
from oracle import lba_exact as ex

FORMATS = [(7, 4, 10), (7, 4, 12), (7, 4, 8), (4, 3, 5), (10, 5, 16), (4, 4, -4), (6, 6, 44), (3, 2, 1), (23, 8, 127)]


def _rows(path):
    with open(path) as fh:
        for line in fh:
            line = line.strip()
            if line and not line.startswith("#"):
                yield line.split()


def test_range_closed_forms(golden_dir):
    n = 0
    for M, E, b, r_of, r_uf in _rows(os.path.join(golden_dir, "eq2_ranges.txt")):
        fmt = (int(M), int(E), int(b), 0, 1)
        got_of, got_uf = orc.fmt_range(fmt)
        assert got_of == float.fromhex(r_of)
        assert got_uf == float.fromhex(r_uf)
        assert ex.r_of(*fmt[:3]) == Fraction(float.fromhex(r_of))
        n += 1
    assert n == 6


def test_bit_count_and_default_bias():
    # B = M + E + 1 ; the paper's accumulator M7E4 is 12 bits and its default bias is 2^(E-1) = 8
    assert 7 + 4 + 1 == 12
    # with b = 2^(E-1) the representable binades are [-b, 2^E - b - 1]: R_OF just under 2^(2^E - b)
    r_of, r_uf = orc.fmt_range((7, 4, 8, 0, 1))
    assert r_uf == 2.0 ** -8 and 2.0 ** 7 < r_of < 2.0 ** 8


def test_spot_values(golden_dir):
    n = 0
    for M, E, b, rnd, flags, x, want in _rows(os.path.join(golden_dir, "eq2_spot_values.txt")):
        fmt = (int(M), int(E), int(b), int(rnd), int(flags))
        assert orc.quantise(fmt, float(x)) == float(want), (fmt, x)
        assert ex.quantise(fmt, Fraction(float(x))) == Fraction(float(want)), (fmt, x)
        n += 1
    assert n == 17


def _random_doubles(rng, fmt, n):
    M, E, b = fmt
    lo, hi = -b - 3, 2 ** E - b + 2
    mag = np.exp2(rng.uniform(lo, hi, n))
    return mag * rng.choice([-1.0, 1.0], n)


@pytest.mark.parametrize("rounding", [0, 1])
@pytest.mark.parametrize("fmt", FORMATS)
def test_two_codings_agree(fmt, rounding):
    rng = np.random.default_rng(7 + fmt[0] * 100 + fmt[1] * 10 + rounding)
    for flags in (1, 0):
        f = fmt + (rounding, flags)
        for x in _random_doubles(rng, fmt, 300):
            assert Fraction(orc.quantise(f, x)) == ex.quantise(f, Fraction(x))


@pytest.mark.parametrize("rounding", [0, 1])
@pytest.mark.parametrize("fmt", FORMATS[:8])
def test_invariants(fmt, rounding):
    M, E, b = fmt
    f = fmt + (rounding, 1)
    r_of, r_uf = orc.fmt_range(f)
    rng = np.random.default_rng(99 + M + 7 * E + rounding)
    xs = np.sort(_random_doubles(rng, fmt, 2000))
    qs = np.array([orc.quantise(f, x) for x in xs])
    # monotone non-decreasing, odd, idempotent
    assert np.all(np.diff(qs) >= 0)
    for x, q in zip(xs[::20], qs[::20]):
        assert orc.quantise(f, -x) == -q or q == 0
        assert orc.quantise(f, q) == q
    for x, q in zip(xs, qs):
        a = abs(x)
        if a >= r_of:
            assert abs(q) == r_of                      # overflow saturates (Eq. 2, first case)
        elif a < r_uf:
            assert q == 0.0 and not np.signbit(q)      # underflow flushes to +0 (second case)
        else:
            e = np.floor(np.log2(a))
            if rounding == 0:
                assert abs(q) <= a and a - abs(q) < 2.0 ** (e - M)     # Table 1: swamping error bound
            else:
                assert abs(abs(q) - a) <= 2.0 ** (e - M - 1)
            # the result lies on the grid of its binade and inside the range
            assert r_uf <= abs(q) <= r_of
            steps = abs(q) / 2.0 ** (np.floor(np.log2(abs(q))) - M)
            assert steps == np.floor(steps)


def test_every_representable_value_is_a_fixed_point():
    M, E, b = 4, 3, 5
    for rounding in (0, 1):
        f = (M, E, b, rounding, 1)
        values = [2.0 ** e * (1 + m / 2 ** M) for e in range(-b, 2 ** E - b) for m in range(2 ** M)]
        assert len(values) == 2 ** (M + E)
        for v in values:
            assert orc.quantise(f, v) == v and orc.quantise(f, -v) == -v
        # between neighbours floor returns the lower one, nearest the closer one
        for lo, hi in zip(values[:-1], values[1:]):
            x = lo + 0.75 * (hi - lo)
            assert orc.quantise(f, x) == (lo if rounding == 0 else hi)
            assert orc.quantise(f, -x) == (-lo if rounding == 0 else -hi)


def test_nearest_matches_ieee_conversions():
    rng = np.random.default_rng(5)
    # binary32: M=23, E=8; R_UF = 2^-126 needs b = 126 (top binade then 129: unreachable here)
    xs = rng.standard_normal(4000) * np.exp2(rng.integers(-40, 40, 4000))
    f32 = (23, 8, 126, 1, 1)
    for x in xs:
        assert orc.quantise(f32, x) == float(np.float32(x))
    # binary16 inside its normal range: M=10, E=5, R_UF = 2^-14
    f16 = (10, 5, 14, 1, 1)
    xs = rng.uniform(2.0 ** -14, 65000.0, 4000) * rng.choice([-1.0, 1.0], 4000)
    for x in xs:
        assert orc.quantise(f16, x) == float(np.float16(x))
    # bfloat16 via PyTorch: M=7, E=8
    bf16 = (7, 8, 126, 1, 1)
    xs = (rng.standard_normal(4000) * np.exp2(rng.integers(-30, 30, 4000))).astype(np.float32)
    want = torch.from_numpy(xs).to(torch.bfloat16).to(torch.float64).numpy()
    for x, wv in zip(xs, want):
        assert orc.quantise(bf16, float(x)) == wv


def test_floor_matches_truncated_ieee_conversion():
    rng = np.random.default_rng(6)
    f32 = (23, 8, 126, 0, 1)
    xs = rng.standard_normal(4000) * np.exp2(rng.integers(-40, 40, 4000))
    for x in xs:
        t = np.float32(x)
        if abs(float(t)) > abs(x):                       # nearest went away from zero: step back
            t = np.nextafter(t, np.float32(0.0))
        assert orc.quantise(f32, x) == float(t)
    # bfloat16 truncation is a 16-bit mask on the binary32 pattern
    bf16 = (7, 8, 126, 0, 1)
    xs32 = xs.astype(np.float32)
    masked = (xs32.view(np.uint32) & np.uint32(0xFFFF0000)).view(np.float32)
    for x, wv in zip(xs32, masked):
        assert orc.quantise(bf16, float(x)) == float(wv)


def test_full_swamping_rule():
    # Sec. 2.3: |z1| > 2^(M+1) |z2|  =>  Q(z1 + z2) = z1.  With the paper's floor rounding the bound
    # is exactly "z2 is less than one grid step of z1": it holds for equal signs, and with opposite
    # signs floor returns the grid point below z1.  Nearest-even swamps only below half a step.
    M, E, b = 7, 4, 10
    rng = np.random.default_rng(11)
    for _ in range(500):
        e = int(rng.integers(-b + 1, 2 ** E - b - 1))
        z1 = 2.0 ** e * (1 + int(rng.integers(1, 2 ** M)) / 2 ** M)
        z2 = z1 / 2 ** (M + 1) * float(rng.uniform(0.01, 0.99))
        assert abs(z1) > 2 ** (M + 1) * abs(z2)
        assert orc.quantise((M, E, b, 0, 1), z1 + z2) == z1
        assert orc.quantise((M, E, b, 0, 1), -z1 - z2) == -z1
        assert orc.quantise((M, E, b, 0, 1), z1 - z2) == z1 - 2.0 ** (e - M)
        z3 = 2.0 ** (e - M - 1) * float(rng.uniform(0.01, 0.99))
        assert orc.quantise((M, E, b, 1, 1), z1 + z3) == z1
        assert orc.quantise((M, E, b, 1, 1), z1 - z3) == z1
    # one step beyond the bound the addend is no longer swamped
    z1 = 1.5
    assert orc.quantise((M, E, b, 0, 1), z1 + z1 / 2 ** (M + 1) * 2) > z1


def test_no_underflow_flag_keeps_small_values():
    f_on, f_off = (7, 4, 10, 0, 1), (7, 4, 10, 0, 0)
    x = 2.0 ** -13 * 1.3
    assert orc.quantise(f_on, x) == 0.0
    q = orc.quantise(f_off, x)
    assert 0 < q <= x and x - q < 2.0 ** (-13 - 7)


def test_format_errors():
    with pytest.raises(orc.OracleError):
        orc.quantise((0, 4, 8, 0, 1), 1.0)
    with pytest.raises(orc.OracleError):
        orc.quantise((7, 4, 8, 2, 1), 1.0)
    with pytest.raises(orc.OracleError):
        orc.quantise((7, 11, 8, 0, 1), 1.0)          # (E = 0 is no error any more: it selects Eq. 1)


# ---------------------------------------------------------------- Eq. 1: the fixed-point quantiser
def test_fixed_point_hand_worked_values(golden_dir):
    for B, b, wrap, x, want in _rows(os.path.join(golden_dir, "eq1_fixed_point.txt")):
        fmt = (int(B), 0, int(b), 0, 2 if wrap == "1" else 0)
        assert orc.quantise(fmt, float(x)) == float(want), (fmt, x)
        assert ex.quantise(fmt, Fraction(x)) == Fraction(want), (fmt, x)


def test_fixed_point_range_closed_forms_and_invariants():
    rng = np.random.default_rng(3)
    for B, b in ((8, 0), (12, 4), (8, 2), (6, -2), (16, 7), (24, 5)):
        lo, hi = ex.fixed_range(B, b)
        assert lo == -Fraction(2) ** (B - b - 1) and hi == Fraction(2 ** (B - 1) - 1, 1) / Fraction(2) ** b
        fmt = (B, 0, b, 0, 0)
        assert orc.quantise(fmt, 1e30) == float(hi) and orc.quantise(fmt, -1e30) == float(lo)
        xs = np.sort(rng.uniform(float(lo) * 1.2, float(hi) * 1.2, 400))
        ys = np.array([orc.quantise(fmt, float(x)) for x in xs])
        assert (np.diff(ys) >= 0).all()                                   # monotone
        assert all(orc.quantise(fmt, float(y)) == y for y in ys)          # idempotent
        inside = (xs > float(lo)) & (xs < float(hi))
        err = xs[inside] - ys[inside]
        assert (err >= 0).all() and (err < 2.0 ** -b).all()               # floor: 0 <= x - Q(x) < 2^-b
        assert all(float(ex.quantise(fmt, Fraction(float(x)))) == y for x, y in zip(xs, ys))
        # wrap-around agrees with saturation inside the range and is periodic with period 2^(B-b)
        wfmt = (B, 0, b, 0, 2)
        for x in xs[inside][::20]:
            assert orc.quantise(wfmt, float(x)) == orc.quantise(fmt, float(x))
            assert orc.quantise(wfmt, float(x) + 2.0 ** (B - b)) == orc.quantise(fmt, float(x))


def test_fixed_point_integer_accumulator_against_numpy_integers():
    # b = 0: Q is integer arithmetic.  Saturation: a Python-integer loop with a clamp after every addition.
    # Wrap-around: reduction modulo 2^B is a ring homomorphism, so the result is the exact integer dot product
    # wrapped once, whatever the order of accumulation.
    from paper_2401_14110_b200 import synth
    A = synth.small_integer_codes((6, 70), 21, max_abs=15).numpy()
    Bm = synth.small_integer_codes((5, 70), 22, max_abs=15).numpy()
    av = synth.e4m3_decode(torch.from_numpy(A)).numpy().astype(np.int64)
    bv = synth.e4m3_decode(torch.from_numpy(Bm)).numpy().astype(np.int64)
    one = np.ones(1, np.float32)
    exact = av @ bv.T
    for Bbits in (8, 10, 12, 16):
        lo, hi = -(1 << (Bbits - 1)), (1 << (Bbits - 1)) - 1
        sat = (Bbits, 0, 0, 0, 0)
        got = orc.gemm(A, Bm, one, one, None, (16, 0, 0, 0, 0), sat, 0, 1)
        want = np.zeros_like(exact)
        for m in range(6):
            for n in range(5):
                s = 0
                for k in range(70):
                    s = min(max(s + int(av[m, k] * bv[n, k]), lo), hi)
                want[m, n] = s
        assert (got == want).all()
        wrap = (Bbits, 0, 0, 0, 2)
        wrapped = (exact - lo) % (1 << Bbits) + lo
        for order, chunk in ((0, 1), (1, 16), (1, 7)):
            assert (orc.gemm(A, Bm, one, one, None, wrap, wrap, order, chunk) == wrapped).all()
    assert (np.abs(exact) > 127).any() and (np.abs(exact) < 2047).all()


def test_fixed_point_chain_against_exact_rationals():
    rng = np.random.default_rng(8)
    finite = np.array([c for c in range(256) if (c & 0x7F) != 0x7F], np.uint8)
    one = np.ones(1, np.float32)
    for trial in range(30):
        K = int(rng.integers(1, 50))
        x = finite[rng.integers(0, finite.size, K)]
        w = finite[rng.integers(0, finite.size, K)]
        pf = (int(rng.integers(10, 25)), 0, int(rng.integers(-2, 9)), 0, 2 * (trial % 2))
        af = (int(rng.integers(8, 25)), 0, int(rng.integers(-4, 7)), 0, 2 * (trial % 2))
        order, chunk = [(0, 1), (1, 16), (1, 5)][trial % 3]
        got = orc.gemm(x[None], w[None], one, one, None, pf, af, order, chunk)[0, 0]
        assert Fraction(float(got)) == ex.dot(pf, af, order, chunk, x, w)


def test_fixed_point_format_errors():
    for bad in ((1, 0, 0, 0, 0), (33, 0, 0, 0, 0), (8, 0, 0, 1, 0), (8, 0, 100, 0, 0)):
        with pytest.raises(orc.OracleError):
            orc.quantise(bad, 1.0)
    x = np.full((1, 4), 0x48, np.uint8)
    with pytest.raises(orc.OracleError):     # the estimators are defined for the floating-point accumulator
        orc.gemm_last_overflow(x, x, (12, 0, 0, 0, 0), (12, 0, 0, 0, 0))
