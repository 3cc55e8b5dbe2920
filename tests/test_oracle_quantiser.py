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
        orc.quantise((7, 0, 8, 0, 1), 1.0)
