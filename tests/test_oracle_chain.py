"""Pins for the oracle's FMAq chain (Eq. 4, Eq. 8-9, chunked accumulation).  CPU only."""
import ctypes
import os
import subprocess
from fractions import Fraction

import numpy as np
import pytest
import torch

from oracle import lba_oracle as orc
from oracle import lba_exact as ex
from paper_2401_14110_b200 import synth

SEQ, CHK = orc.SEQUENTIAL, orc.CHUNKED
WIDE_NEAREST = (23, 8, 127, 1, 1)
WIDE_FLOOR = (23, 8, 127, 0, 1)
FINITE = np.array([c for c in range(256) if (c & 0x7F) != 0x7F], dtype=np.uint8)


def _decode_f32(codes):
    return synth.e4m3_decode(torch.from_numpy(np.ascontiguousarray(codes))).numpy()


def test_decode_matches_pytorch_float8_cast():
    vals = _decode_f32(FINITE)
    for c, v in zip(FINITE, vals):
        assert orc.decode_e4m3(int(c)) == float(v)
        assert ex.decode_e4m3(int(c)) == Fraction(float(v))
    assert orc.decode_e4m3(0x7E) == 448.0 and orc.decode_e4m3(0x01) == 2.0 ** -9
    for nan_code in (0x7F, 0xFF):
        with pytest.raises(orc.OracleError):
            orc.decode_e4m3(nan_code)


def test_hand_worked_chains(golden_dir):
    n = 0
    with open(os.path.join(golden_dir, "fmaq_chains.txt")) as fh:
        for line in fh:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            name, rnd, order, chunk, K, xb, wb, want, *sums = line.split()
            rnd, order, chunk, K = int(rnd), int(order), int(chunk), int(K)
            prod, acc = (7, 4, 12, rnd, 1), (7, 4, 10, rnd, 1)
            x = np.full(K, int(xb, 16), np.uint8)
            w = np.full(K, int(wb, 16), np.uint8)
            y, tr = orc.dot(prod, acc, order, chunk, x, w, trace=True)
            assert y == float(want), name
            if sums:
                assert list(tr) == [float(v) for v in sums], name
            assert ex.dot(prod, acc, order, chunk, x, w) == Fraction(float(want)), name
            n += 1
    assert n == 6


@pytest.fixture(scope="module")
def fp32_chain(tmp_path_factory):
    src = os.path.join(os.path.dirname(__file__), "helpers", "fp32_chain.c")
    lib = str(tmp_path_factory.mktemp("fp32") / "libfp32_chain.so")
    subprocess.run(["gcc", "-O1", "-frounding-math", "-ffp-contract=off", "-fPIC", "-shared", src, "-o", lib, "-lm"],
                   check=True)
    dll = ctypes.CDLL(lib)
    dll.fp32_chain.restype = ctypes.c_float
    dll.fp32_chain.argtypes = [ctypes.POINTER(ctypes.c_float), ctypes.POINTER(ctypes.c_float), ctypes.c_int64,
                               ctypes.c_int]

    def run(x, w, toward_zero):
        x = np.ascontiguousarray(x, np.float32)
        w = np.ascontiguousarray(w, np.float32)
        return float(dll.fp32_chain(x.ctypes.data_as(ctypes.POINTER(ctypes.c_float)),
                                    w.ctypes.data_as(ctypes.POINTER(ctypes.c_float)), len(x), int(toward_zero)))
    return run


@pytest.mark.parametrize("K", [1, 7, 64, 577, 3000])
def test_wide_accumulator_is_ieee_binary32_summation(fp32_chain, K):
    # (M23, E8, b=127): R_UF = 2^-127 and R_OF > 2^128 cannot be reached from E4M3 products, so
    # FMAq is one correctly rounded binary32 addition per step (Eq. 4 with Q = binary32 rounding).
    for trial in range(4):
        x = synth.random_codes((K,), 100 + trial).numpy()
        w = synth.random_codes((K,), 200 + trial).numpy()
        xf, wf = _decode_f32(x), _decode_f32(w)
        s = np.float32(0)
        for a, b in zip(xf, wf):
            s = np.float32(s + np.float32(a * b))
        assert orc.dot(WIDE_NEAREST, WIDE_NEAREST, SEQ, 16, x, w) == float(s)
        assert fp32_chain(xf, wf, False) == float(s)
        assert orc.dot(WIDE_FLOOR, WIDE_FLOOR, SEQ, 16, x, w) == fp32_chain(xf, wf, True)


def test_chunk_extremes_equal_sequential():
    prod, acc = (7, 4, -2, 0, 1), (7, 4, -4, 0, 1)
    for K in (1, 5, 16, 17, 100):
        x = synth.random_codes((K,), 31 + K).numpy()
        w = synth.random_codes((K,), 41 + K).numpy()
        seq = orc.dot(prod, acc, SEQ, 16, x, w)
        assert orc.dot(prod, acc, CHK, K, x, w) == seq          # one chunk: second level adds 0
        assert orc.dot(prod, acc, CHK, K + 5, x, w) == seq
        # chunks of one compute Q_acc(Q_acc(P) + T): the same as sequential whenever Q_acc leaves a
        # lone product unchanged, e.g. when both quantisers share one format
        same = (7, 4, -2, 0, 1)
        assert orc.dot(same, same, CHK, 1, x, w) == orc.dot(same, same, SEQ, 16, x, w)


def test_order_is_observable():
    # Sec. 3 / App. D: accumulation order changes the result because of swamping
    prod, acc = (7, 4, -2, 0, 1), (7, 4, -4, 0, 1)
    differ = 0
    for t in range(20):
        a, _, b, _ = synth.gemm_case(1, 1, 576, 900 + t)
        differ += orc.dot(prod, acc, SEQ, 16, a[0].numpy(), b[0].numpy()) != orc.dot(prod, acc, CHK, 16, a[0].numpy(),
                                                                                       b[0].numpy())
    assert differ > 0


@pytest.mark.parametrize("order,chunk", [(SEQ, 16), (CHK, 16), (CHK, 5)])
def test_exact_when_all_partial_sums_are_representable(order, chunk):
    # small integers, 10-bit mantissa, wide range: nothing is ever rounded, so the result is the integer dot product
    prod, acc = (10, 6, 20, 0, 1), (10, 6, 20, 0, 1)
    for t in range(10):
        x = synth.small_integer_codes((40,), 300 + t, max_abs=5)
        w = synth.small_integer_codes((40,), 400 + t, max_abs=5)
        want = int(np.dot(_decode_f32(x.numpy()).astype(np.int64), _decode_f32(w.numpy()).astype(np.int64)))
        assert abs(want) < 1024
        assert orc.dot(prod, acc, order, chunk, x.numpy(), w.numpy()) == float(want)


def test_zero_products_leave_the_sum_unchanged():
    # FMAq(0, w, S) = Q_acc(S) = S: the fact that makes padded convolution taps and K padding harmless
    prod, acc = (7, 4, -2, 0, 1), (7, 4, -4, 0, 1)
    x = synth.random_codes((64,), 1).numpy()
    w = synth.random_codes((64,), 2).numpy()
    base = orc.dot(prod, acc, SEQ, 16, x, w)
    xz = np.concatenate([x, np.zeros(9, np.uint8), np.full(3, 0x80, np.uint8)])
    wz = np.concatenate([w, synth.random_codes((12,), 3).numpy()])
    assert orc.dot(prod, acc, SEQ, 16, xz, wz) == base


FORMAT_PAIRS = [((7, 4, -2), (7, 4, -4)), ((7, 4, 12), (7, 4, 10)), ((4, 4, -2), (4, 4, -4)), ((5, 5, 14), (5, 5, 12)),
                ((10, 6, 46), (10, 6, 44)), ((4, 3, 5), (4, 3, 5)), ((3, 4, 2), (9, 5, 9))]


def _unit(prod, acc):
    # counts of 2^-U with U even: operands are counts of 2^-(U/2); room for two quantisations of a cancelled sum
    return 2 * max(9, (18 + 2 * max(prod[0], acc[0]) + 1) // 2)


def _grid_values(fmt):
    """Every non-negative value of Q^FLOAT_{M,E,b} (Eq. 2): 0 and 2^e (1 + n/2^M), as floats (exact for these formats)."""
    M, E, b = fmt[:3]
    return [0.0] + [2.0 ** e * (1 + n / 2.0 ** M) for e in range(-b, 2 ** E - b) for n in range(2 ** M)]


@pytest.mark.parametrize("rounding", [0, 1])
@pytest.mark.parametrize("flags", [1, 0])
def test_brute_force_all_pairs_k1(rounding, flags):
    # every finite E4M3 pair through one FMAq from S = 0, for every format pair, both roundings, with and without
    # the underflow branch: the C++ oracle against the 64-bit integer coding (all pairs) and against the
    # exact-rational coding (a third of the pairs)
    from helpers import int_coding as ic
    codes = FINITE
    vals = [ex.decode_e4m3(int(c)) for c in codes]
    for pf, af in FORMAT_PAIRS:
        prod, acc = pf + (rounding, flags), af + (rounding, flags)
        U = _unit(prod, acc)
        got = orc.fmaq_grid(prod, acc, codes, codes, [0.0])[0]           # got[i][j] = FMAq(c_i, c_j, 0)
        xi = np.array([ic.e4m3_int(int(c), U // 2) for c in codes], dtype=np.int64)
        want = ic.fmaq_int(prod, acc, xi[:, None], xi[None, :], 0, U)
        assert np.array_equal(np.ldexp(want.astype(np.float64), -U), got), (prod, acc)
        for i in range(len(codes)):
            for j in range(i % 3, len(codes), 3):
                assert Fraction(float(got[i, j])) == ex.quantise(acc, ex.quantise(prod, vals[i] * vals[j])), (pf, af, i, j)
    # the same table through the GEMM entry point (what the GPU parity test of all pairs compares with)
    prod, acc = FORMAT_PAIRS[0][0] + (rounding, flags), FORMAT_PAIRS[0][1] + (rounding, flags)
    out = orc.gemm(codes[:, None], codes[:, None], 1.0, 1.0, None, prod, acc, SEQ, 16)
    assert np.array_equal(out.astype(np.float64), orc.fmaq_grid(prod, acc, codes, codes, [0.0])[0])


@pytest.mark.parametrize("rounding", [0, 1])
def test_last_step_of_any_short_chain_from_a_covering_set_of_running_sums(rounding):
    # A chain of K <= 4 steps is K FMAq steps, each from a running sum S that lies on the accumulator's grid.  Instead
    # of all 254^(2K) chains (4e9 already at K = 2), every code pair is run as one step from a covering set of S:
    # 0, the grid values of the lowest and of the highest binade (all of them up to M = 6, 64 of each above), +-R_OF, the values just above R_UF, and every
    # 16th grid value in between (a coarser stride for the larger grids), both signs (for the 8-bit accumulator of
    # Sec. 4: the whole grid).  C++ oracle
    # against the 64-bit integer coding, element by element.
    from helpers import int_coding as ic
    codes = FINITE
    for pf, af in FORMAT_PAIRS:
        prod, acc = pf + (rounding, 1), af + (rounding, 1)
        U = _unit(prod, acc)
        grid = _grid_values(acc)
        per = 2 ** acc[0]
        st = max(1, per // 64)
        pick = set(grid[:1 + per:st]) | set(grid[-per::st]) | set(grid[1::max(16, len(grid) // 96)]) | {grid[-1], grid[1], grid[2]}
        if len(grid) <= 600:
            pick = set(grid)
        s_vals = sorted(pick | {-v for v in pick})
        # sums of products are multiples of 2^-18 at least: grid values finer than the integer unit cannot occur in a chain
        s_vals = [v for v in s_vals if (Fraction(v) * 2 ** U).denominator == 1 and (v == 0 or abs(v) >= 2.0 ** -18)]
        s_int = np.array([int(Fraction(v) * 2 ** U) for v in s_vals], dtype=np.int64)
        xi = np.array([ic.e4m3_int(int(c), U // 2) for c in codes], dtype=np.int64)
        for lo in range(0, len(s_vals), 64):
            got = orc.fmaq_grid(prod, acc, codes, codes, s_vals[lo:lo + 64])
            want = ic.fmaq_int(prod, acc, xi[None, :, None], xi[None, None, :], s_int[lo:lo + 64, None, None], U)
            assert np.array_equal(np.ldexp(want.astype(np.float64), -U), got), (prod, acc, lo)


def test_integer_coding_agrees_with_rationals_on_whole_chains_for_e4():
    # for E = 4 every value is a count of 2^-(b+M) below 2^(16-b): a chain in plain integers, against the C++ chain
    from helpers import int_coding as ic
    rng = np.random.default_rng(77)
    for (pf, af) in [FORMAT_PAIRS[0], FORMAT_PAIRS[1], FORMAT_PAIRS[2]]:
        for rounding in (0, 1):
            prod, acc = pf + (rounding, 1), af + (rounding, 1)
            U = _unit(prod, acc)
            for trial in range(30):
                K = int(rng.integers(1, 80))
                x = rng.choice(FINITE, K)
                w = rng.choice(FINITE, K)
                xs = [ic.e4m3_int(int(c), U // 2) for c in x]
                ws = [ic.e4m3_int(int(c), U // 2) for c in w]
                s = np.int64(0)
                for a_, b_ in zip(xs, ws):                         # Eq. 8-9
                    s = ic.fmaq_int(prod, acc, a_, b_, s, U)
                assert abs(int(s)) < 2 ** 62
                assert float(np.ldexp(float(s), -U)) == orc.dot(prod, acc, SEQ, 1, x, w)
                t = np.int64(0)                                    # two hierarchies, chunk 16
                for j in range(0, K, 16):
                    c = np.int64(0)
                    for a_, b_ in zip(xs[j:j + 16], ws[j:j + 16]):
                        c = ic.fmaq_int(prod, acc, a_, b_, c, U)
                    t = ic.quantise_int(c + t, *acc, U)
                assert float(np.ldexp(float(t), -U)) == orc.dot(prod, acc, CHK, 16, x, w)


@pytest.mark.parametrize("rounding", [0, 1])
@pytest.mark.parametrize("K", [2, 3, 4, 33])
def test_sampled_chains_against_exact_rationals(K, rounding):
    for fi, (pf, af) in enumerate(FORMAT_PAIRS):
        for flags in (1, 0):
            prod, acc = pf + (rounding, flags), af + (rounding, flags)
            for t in range(25 if K <= 4 else 6):
                x = synth.random_codes((K,), 5000 + 97 * fi + t).numpy()
                w = synth.random_codes((K,), 6000 + 89 * fi + t).numpy()
                for order, chunk in ((SEQ, 16), (CHK, 16), (CHK, 2)):
                    got = orc.dot(prod, acc, order, chunk, x, w)
                    assert Fraction(got) == ex.dot(prod, acc, order, chunk, x, w), (prod, acc, order, chunk, t)


def test_planted_mistakes_are_caught_by_the_pins():
    """Each plausible slip, applied to the exact-rational coding, must break a hand-worked value."""
    x = [ex.decode_e4m3(0x48)] * 5
    prod, acc = (7, 4, 12, 0, 1), (7, 4, 10, 0, 1)

    def chain(q_prod, q_acc, n=5):
        s = Fraction(0)
        for a in x[:n]:
            s = q_acc(q_prod(a * a) + s)
        return s
    good = chain(lambda v: ex.quantise(prod, v), lambda v: ex.quantise(acc, v))
    assert good == Fraction(63.75)
    # dropped Q_prod
    assert chain(lambda v: v, lambda v: ex.quantise(acc, v), 3) != Fraction(47.75)
    # Q_acc applied only at the end of the sum instead of after every addition
    s3 = sum(ex.quantise(prod, a * a) for a in x[:3])
    s4 = ex.quantise(acc, s3 + ex.quantise(prod, x[3] * x[3]))
    assert s4 != Fraction(63.5)          # 47.8125 + 15.9375 = 63.75 exactly; per-step rounding gives 63.5
    # biases swapped
    assert chain(lambda v: ex.quantise(acc, v), lambda v: ex.quantise(prod, v), 2) != Fraction(31.875)
    # nearest instead of floor
    assert chain(lambda v: ex.quantise(prod, v), lambda v: ex.quantise((7, 4, 10, 1, 1), v), 4) != Fraction(63.5)
    # last product dropped (the S_{N-1} misprint of Eq. 8-9)
    assert chain(lambda v: ex.quantise(prod, v), lambda v: ex.quantise(acc, v), 4) != good


def test_last_overflow_index_hand_worked_and_against_exact_rationals():
    # chain A of the golden file: x = w = 4.0, products saturate Q_prod to 15.9375; the accumulator input is
    # 15.9375, 31.875, 47.8125, 63.6875 (all below R_OF_acc = 63.75), then 63.5 + 15.9375 = 79.4375 >= 63.75 at
    # step 4 and at every later step (S stays at 63.75)
    prod, acc = (7, 4, 12, 0, 1), (7, 4, 10, 0, 1)
    for K, want in ((1, -1), (4, -1), (5, 4), (7, 6)):
        x = np.full((1, K), 0x48, np.uint8)
        assert orc.gemm_last_overflow(x, x, prod, acc)[0, 0] == want
        assert ex.last_overflow(prod, acc, x[0], x[0]) == want
    # a negative tail brings the sum back below R_OF: the last overflow stays where it was
    x = np.array([[0x48] * 6 + [0xC8] * 3], np.uint8)      # six times +4, three times -4
    w = np.full((1, 9), 0x48, np.uint8)
    assert orc.gemm_last_overflow(x, w, prod, acc)[0, 0] == 5
    # a step that adds nothing while S sits at R_OF still has |0 + S| >= R_OF
    x = np.array([[0x48] * 6 + [0x00] * 2], np.uint8)
    assert orc.gemm_last_overflow(x, np.full((1, 8), 0x48, np.uint8), prod, acc)[0, 0] == 7
    # random small cases against the exact-rational restatement of Eq. 2 / Eq. 4
    rng = np.random.default_rng(5)
    finite = np.array([c for c in range(256) if (c & 0x7F) != 0x7F], np.uint8)
    hits = 0
    for trial in range(60):
        K = int(rng.integers(1, 40))
        A = finite[rng.integers(0, finite.size, (3, K))]
        B = finite[rng.integers(0, finite.size, (2, K))]
        if trial % 2:
            A, B = A & 0x7F, B & 0x7F
        fm = [((7, 4, 12, 0, 1), (7, 4, 10, 0, 1)), ((7, 4, -2, 0, 1), (7, 4, -4, 0, 1)), ((4, 4, 0, 0, 0), (5, 4, 2, 0, 0))][trial % 3]
        got = orc.gemm_last_overflow(A, B, fm[0], fm[1])
        for m in range(3):
            for n in range(2):
                want = ex.last_overflow(fm[0], fm[1], A[m], B[n])
                assert got[m, n] == want
                hits += want >= 0
    assert hits > 20


def _bits_of(words, n):
    return [(int(words[i // 32]) >> (i % 32)) & 1 for i in range(n)]


def test_ste_masks_hand_worked_chains():
    prod, acc = (7, 4, 12, 0, 1), (7, 4, 10, 0, 1)
    # x = w = 4.0: the accumulator input is 15.9375, 31.875, 47.8125, 63.6875, then 79.4375 and 79.6875... >= 63.75:
    # STE^OF passes the first four steps only
    x = np.full((1, 7), 0x48, np.uint8)
    m1, m2 = orc.gemm_ste_mask(x, x, prod, acc, 0, 1, orc.STE_OF)
    assert m2 is None and m1.shape == (1, 1, 1) and m1[0, 0, 0] == 0b0001111
    # the stagnation chain (x = 0.5, w = 0.25, product 0.125): every step adds 0.125 exactly until S = 32, where
    # the grid step is 0.25 and the product is swamped: z - S = 0.125 = |x w| for 256 steps, then 0.  STE^DIFF with
    # eps2 = 0.5 therefore passes exactly the first 256 steps; nothing ever overflows, so STE^OF passes all 300
    a = np.full((1, 300), 0x30, np.uint8)
    w = np.full((1, 300), 0x28, np.uint8)
    m1, _ = orc.gemm_ste_mask(a, w, prod, acc, 0, 1, orc.STE_DIFF, 1e-6, 0.5)
    assert m1.shape == (1, 10, 1) and _bits_of(m1[0, :, 0], 300) == [1] * 256 + [0] * 44
    assert (m1[0, 9, 0] >> 12) == 0                                   # unused high bits of the last word
    m1, _ = orc.gemm_ste_mask(a, w, prod, acc, 0, 1, orc.STE_OF)
    assert _bits_of(m1[0, :, 0], 300) == [1] * 300
    # chunks of 16 keep every first-level sum at <= 2.0 and the folds add 2.0 to T <= 37.5 exactly: all bits pass
    m1, m2 = orc.gemm_ste_mask(a, w, prod, acc, 1, 16, orc.STE_DIFF, 1e-6, 0.5)
    assert _bits_of(m1[0, :, 0], 300) == [1] * 300 and _bits_of(m2[0, :, 0], 19) == [1] * 19 and m2.shape == (1, 1, 1)
    # K = 576 in chunks of 16: T climbs by 2.0 per fold and saturates at 63.75 at the 32nd fold (exact sum 64):
    # STE^OF of the folds is 1 for folds 0..30 and 0 from fold 31 on
    a = np.full((1, 576), 0x30, np.uint8)
    w = np.full((1, 576), 0x28, np.uint8)
    m1, m2 = orc.gemm_ste_mask(a, w, prod, acc, 1, 16, orc.STE_OF)
    assert _bits_of(m2[0, :, 0], 36) == [1] * 31 + [0] * 5 and m2.shape == (1, 2, 1)
    assert all(v == 0xFFFFFFFF for v in m1[0, :, 0])
    # a single chunk still has its fold: x = w = 4.0, K = 7, chunk 16: C = 63.75 (saturated), |C + 0| >= R_OF
    x = np.full((1, 7), 0x48, np.uint8)
    m1, m2 = orc.gemm_ste_mask(x, x, prod, acc, 1, 16, orc.STE_OF)
    assert m1[0, 0, 0] == 0b0001111 and m2[0, 0, 0] == 0
    # a zero product never passes STE^DIFF (App. D sets alpha = 0 there): z = S
    x = np.array([[0x48, 0x00, 0x48]], np.uint8)
    m1, _ = orc.gemm_ste_mask(x, np.full((1, 3), 0x48, np.uint8), prod, acc, 0, 1, orc.STE_DIFF, 1e-6, 0.01)
    assert m1[0, 0, 0] == 0b101


def test_ste_masks_against_exact_rationals_and_last_overflow():
    rng = np.random.default_rng(11)
    finite = np.array([c for c in range(256) if (c & 0x7F) != 0x7F], np.uint8)
    fmts = [((7, 4, 12, 0, 1), (7, 4, 10, 0, 1)), ((7, 4, -2, 0, 1), (7, 4, -4, 0, 1)), ((4, 4, 0, 0, 0), (5, 4, 2, 0, 0)),
            ((4, 3, 5, 0, 1), (4, 3, 5, 0, 1))]
    zeros = ones = 0
    for trial in range(48):
        K = int(rng.integers(1, 90))
        A = finite[rng.integers(0, finite.size, (2, K))]
        B = finite[rng.integers(0, finite.size, (2, K))]
        if trial % 2:
            A, B = A & 0x7F, B & 0x7F
        pf, af = fmts[trial % 4]
        order, chunk = [(0, 1), (1, 16), (1, 5), (1, 32), (1, 100)][trial % 5]
        for kind, name, e1, e2 in ((orc.STE_OF, "OF", 0.0, 0.0), (orc.STE_DIFF, "DIFF", 2.0 ** -20, 0.25),
                                   (orc.STE_DIFF, "DIFF", 1e-3, 0.9)):
            m1, m2 = orc.gemm_ste_mask(A, B, pf, af, order, chunk, kind, e1, e2)
            for m in range(2):
                for n in range(2):
                    f, s = ex.ste_bits(pf, af, order, chunk, A[m], B[n], name, e1, e2)
                    assert _bits_of(m1[m, :, n], K) == f
                    assert order == 0 or _bits_of(m2[m, :, n], len(s)) == s
                    zeros += f.count(0)
                    ones += f.count(1)
                    if kind == orc.STE_OF and order == 0:
                        # the last-overflow index is the position of the highest 0 bit of the sequential OF mask
                        want = max((i for i, b in enumerate(f) if b == 0), default=-1)
                        assert orc.gemm_last_overflow(A[m:m + 1], B[n:n + 1], pf, af)[0, 0] == want
    assert zeros > 500 and ones > 500
