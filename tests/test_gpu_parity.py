"""CUDA path versus the CPU oracle, bit for bit, through the C ABI.  Needs a B200."""
import numpy as np
import pytest
import torch

from oracle import lba_oracle as orc
from paper_2401_14110_b200 import binding as lba
from helpers.fmt_range import r_of, r_uf
from paper_2401_14110_b200 import synth
from paper_2401_14110_b200 import m4e3_input_formats, FLAG_INPUT_M4E3
from paper_2401_14110_b200 import (LbaFormat, fixed_point_format, code_domain_formats, M7E4_PAPER, WIDE, ORDER_SEQUENTIAL as SEQ,
                                   ORDER_CHUNKED as CHK)

pytestmark = pytest.mark.gpu

DEV = "cuda:0"


def _bits(a):
    return np.ascontiguousarray(a, dtype=np.float32).view(np.uint32)


def assert_bit_equal(got, want, what=""):
    got = got.detach().cpu().numpy() if isinstance(got, torch.Tensor) else got
    g, w = _bits(got).reshape(-1), _bits(want).reshape(-1)
    bad = np.nonzero(g != w)[0]
    assert bad.size == 0, (f"{what}: {bad.size} of {g.size} outputs differ; first at {bad[0]}: "
                           f"gpu={got.reshape(-1)[bad[0]]!r} oracle={np.asarray(want).reshape(-1)[bad[0]]!r}")


def gpu_gemm(A, B, sa, sb, bias, prod, acc, order, chunk):
    d = lambda t: None if t is None else t.to(DEV)
    return lba.lba_gemm(d(A), d(B), d(sa), d(sb), d(bias), prod, acc, order, chunk)


def ref_gemm(A, B, sa, sb, bias, prod, acc, order, chunk):
    n = lambda t: None if t is None else t.numpy()
    return orc.gemm(n(A), n(B), n(sa), n(sb), n(bias), prod.as_tuple(), acc.as_tuple(), order, chunk)


FORMATS = {
    "m7e4_code": code_domain_formats(7, 4),                                   # floor_fast
    "m7e4_paper": M7E4_PAPER,                                                 # Q_prod saturates: floor_full
    "m4e4": code_domain_formats(4, 4),                                        # Q_prod rounds
    "m10e5": code_domain_formats(10, 5),
    "m5e6": code_domain_formats(5, 6),
    "m8e6": code_domain_formats(8, 6),                                        # no product can be cut or flushed: fused product and sum
    "m4e3_mnist": (LbaFormat(4, 3, 5), LbaFormat(4, 3, 5)),                   # Sec. 4 accumulator
    "mixed": (LbaFormat(3, 4, 2), LbaFormat(9, 5, 9)),
    "m7e4_code_rne": code_domain_formats(7, 4, rounding=1),
    "m4e4_rne": code_domain_formats(4, 4, rounding=1),
    "m10e6_rne": code_domain_formats(10, 6, rounding=1),
    "m7e4_paper_rne": (LbaFormat(7, 4, 12, 1), LbaFormat(7, 4, 10, 1)),
    "mixed_rne": (LbaFormat(7, 4, -2, 1), LbaFormat(5, 4, -4, 1)),            # products off the accumulator grid
    "m7e4_no_uf": code_domain_formats(7, 4, flags=0),
    "m4e4_rne_no_uf": code_domain_formats(4, 4, rounding=1, flags=0),
    "wide_floor": (WIDE, WIDE),
    "wide_rne": (LbaFormat(23, 8, 127, 1), LbaFormat(23, 8, 127, 1)),
    "m21_rne": (LbaFormat(21, 8, 127, 1), LbaFormat(21, 8, 127, 1)),
}


def test_config1_single_gemm_all_outputs():
    # M = N = 64, K = 576, N(0,1) scaled to absmax 448, M7E4, sequential order
    A, sa, B, sb = synth.gemm_case(64, 64, 576, config=1)
    prod, acc = code_domain_formats(7, 4)
    for order in (SEQ, CHK):
        got = gpu_gemm(A, B, sa, sb, None, prod, acc, order, 16)
        assert_bit_equal(got, ref_gemm(A, B, sa, sb, None, prod, acc, order, 16), f"config 1 order {order}")


@pytest.mark.parametrize("name", list(FORMATS))
def test_all_e4m3_pairs_k1(name):
    # every finite pair through one FMAq: out[i][j] = Q_acc(Q_prod(c_i * c_j))
    prod, acc = FORMATS[name]
    codes = torch.tensor([c for c in range(256) if (c & 0x7F) != 0x7F], dtype=torch.uint8)[:, None].contiguous()
    one = torch.ones(1)
    got = gpu_gemm(codes, codes, one, one, None, prod, acc, SEQ, 16)
    assert_bit_equal(got, ref_gemm(codes, codes, one, one, None, prod, acc, SEQ, 16), name)


@pytest.mark.parametrize("name", list(FORMATS))
@pytest.mark.parametrize("K", [2, 3, 4, 16, 47, 200])
def test_random_codes_short_chains(name, K):
    prod, acc = FORMATS[name]
    A = synth.random_codes((150, K), 10 + K)
    B = synth.random_codes((70, K), 20 + K)
    one = torch.ones(1)
    for order, chunk in ((SEQ, 16), (CHK, 16), (CHK, 3)):
        got = gpu_gemm(A, B, one, one, None, prod, acc, order, chunk)
        assert_bit_equal(got, ref_gemm(A, B, one, one, None, prod, acc, order, chunk), f"{name} K={K} {order}/{chunk}")


@pytest.mark.parametrize("tile", [0, 1, 2, 3])
@pytest.mark.parametrize("name", ["m7e4_code", "m7e4_paper", "m4e4_rne", "wide_rne", "m7e4_no_uf", "m10e6_rne", "m8e6"])
def test_every_tile_shape_with_ragged_edges(tile, name):
    prod, acc = FORMATS[name]
    lba.set_tile_override(tile)
    try:
        for (M, N, K) in ((1, 1, 1), (129, 67, 48), (300, 260, 37), (257, 130, 160)):
            A, sa, B, sb = synth.gemm_case(M, N, K, config=50 + tile)
            sa_rows = torch.linspace(0.5, 1.5, M)
            sb_cols = torch.linspace(0.01, 0.02, N)
            bias = torch.linspace(-1, 1, N)
            for order, chunk in ((SEQ, 16), (CHK, 16), (CHK, 32), (CHK, 5)):
                got = gpu_gemm(A, B, sa_rows, sb_cols, bias, prod, acc, order, chunk)
                assert_bit_equal(got, ref_gemm(A, B, sa_rows, sb_cols, bias, prod, acc, order, chunk),
                                 f"tile {tile} {name} {M}x{N}x{K} {order}/{chunk}")
    finally:
        lba.set_tile_override(-1)


def test_saturation_and_underflow_are_exercised():
    # make sure the parity cases are not vacuous: both special cases of Eq. 2 occur
    prod, acc = code_domain_formats(7, 4)
    A, sa, B, sb = synth.gemm_case(64, 64, 1024, config=7)
    one = torch.ones(1)
    a = synth.e4m3_decode(A).numpy().astype(np.float64)
    b = synth.e4m3_decode(B).numpy().astype(np.float64)
    prods = np.abs(a[0][None, :] * b)
    assert ((prods > 0) & (prods < r_uf(prod))).any()          # products that Q_prod flushes
    # same-sign operands: the running sum climbs to R_OF_acc and stays there
    Apos, Bpos = A & 0x7F, B & 0x7F
    for order in (SEQ, CHK):
        got = gpu_gemm(Apos, Bpos, one, one, None, prod, acc, order, 16).cpu().numpy()
        assert_bit_equal(got, ref_gemm(Apos, Bpos, one, one, None, prod, acc, order, 16))
        assert (got == np.float32(r_of(acc))).any()
        for rname in ("m7e4_code_rne", "m4e4_rne"):      # nearest-even: rounds up into R_OF, never past it
            pr, ar = FORMATS[rname]
            got = gpu_gemm(Apos, Bpos, one, one, None, pr, ar, order, 16).cpu().numpy()
            assert_bit_equal(got, ref_gemm(Apos, Bpos, one, one, None, pr, ar, order, 16), rname)
            assert (got == np.float32(r_of(ar))).any() and (got <= np.float32(r_of(ar))).all()
    # mixed signs around the top: saturate, come back down, saturate negative
    Amix = Apos.clone()
    Amix[:, 512:] |= 0x80
    got = gpu_gemm(Amix, Bpos, one, one, None, prod, acc, CHK, 16).cpu().numpy()
    assert_bit_equal(got, ref_gemm(Amix, Bpos, one, one, None, prod, acc, CHK, 16))


SEARCH_FOUND = [
    # R_OF_acc = 16 - 2^-14 lies off the grid of the products (multiples of 2^-8): a sum that sits at R_OF and meets
    # the product -16 leaves -2^-14, which must not be lost below the carrier's smallest normal number
    (LbaFormat(5, 7, 21, 1, 1 | FLAG_INPUT_M4E3), LbaFormat(17, 5, 28, 1, 1)),
    (LbaFormat(5, 7, 21, 0, 1 | FLAG_INPUT_M4E3), LbaFormat(17, 5, 28, 0, 1)),
    (LbaFormat(12, 6, 30, 0, 1), LbaFormat(21, 5, 31, 0, 1)),
    # Q_prod saturates to R_OF_prod, which has M_prod + 1 significant bits, more than the accumulator keeps: the sum is
    # not one rounding of one binary32 FMA
    (LbaFormat(20, 2, -9, 1, FLAG_INPUT_M4E3), LbaFormat(9, 8, 3, 1, 0)),
    (LbaFormat(19, 3, 8, 1, 1), LbaFormat(8, 6, 34, 1, 1)),
]


@pytest.mark.parametrize("fmts", SEARCH_FOUND, ids=lambda f: "p%d.%d.%d_a%d.%d.%d_r%d" % (f[0].as_tuple()[:3] + f[1].as_tuple()[:4]))
def test_formats_found_by_random_search(fmts):
    prod, acc = fmts
    rng = np.random.default_rng(99)
    finite = np.array([b for b in range(256) if (b & 0x7F) != 0x7F], dtype=np.uint8)
    for (M, N, K) in ((140, 159, 255), (8, 188, 100)):
        A = torch.from_numpy(finite[rng.integers(0, finite.size, (M, K))] & 0x7F)             # one sign
        B = torch.from_numpy(np.where(rng.random((N, K)) < 0.85, 0, finite[rng.integers(0, finite.size, (N, K))]).astype(np.uint8))
        G = synth.gemm_case(M, N, K, config=77)
        one = torch.ones(1)
        for tile in (-1, 0, 3):
            lba.set_tile_override(tile)
            try:
                for order, chunk in ((SEQ, 16), (CHK, 16), (CHK, 32)):
                    for (a, b) in ((A, B), (G[0], B), (G[0], G[2])):
                        got = gpu_gemm(a, b, one, one, None, prod, acc, order, chunk)
                        assert_bit_equal(got, ref_gemm(a, b, one, one, None, prod, acc, order, chunk),
                                         f"{prod} {acc} {M}x{N}x{K} tile {tile} order {order}/{chunk}")
            finally:
                lba.set_tile_override(-1)


@pytest.mark.parametrize("tile", [0, 2, 3])
@pytest.mark.parametrize("name", ["m7e4_code", "m7e4_code_rne", "m4e4_rne", "m10e6_rne", "m7e4_no_uf", "m8e6"])
def test_slow_climb_to_saturation_crosses_every_clamp_decision(tile, name):
    # small same-sign products: each chunk adds a little, so the second-level sum creeps up to R_OF over many
    # chunks.  On the way the kernel's running bound first skips the clamp, then measures the sums, then clamps
    # for good; the sequential order does the same with its first-level bound.  All of it must stay exact, for
    # floor and for nearest-even (whose bound carries the growth of the roundings).
    prod, acc = FORMATS[name]
    M, N, K = 96, 80, 4096
    a = (synth.gaussian((M, K), 81).abs() * 0.25 + 0.05) * torch.linspace(0.2, 1.2, M)[:, None]
    b = synth.gaussian((N, K), 82).abs() * 0.25 + 0.05
    a[:, ::97] *= -1.0                                   # a few negative taps so sums also step back
    A = synth.e4m3_encode(a * 448.0 / 4.0)
    B = synth.e4m3_encode(b * 448.0 / 4.0)
    one = torch.ones(1)
    lba.set_tile_override(tile)
    try:
        for order, chunk in ((CHK, 16), (SEQ, 16), (CHK, 64)):
            got = gpu_gemm(A, B, one, one, None, prod, acc, order, chunk).cpu().numpy()
            assert_bit_equal(got, ref_gemm(A, B, one, one, None, prod, acc, order, chunk), f"{name} tile {tile} {order}/{chunk}")
            if order == CHK and chunk == 16 and name == "m7e4_code":
                frac = float((got == np.float32(r_of(acc))).mean())
                assert 0.02 < frac < 0.98, frac          # some outputs saturate, some do not
    finally:
        lba.set_tile_override(-1)


@pytest.mark.parametrize("case", [
    (24, 128, 128, 64, False),     # attention scores Q K^T: 24 heads, 128 tokens, head size 64
    (24, 128, 64, 128, False),     # attention output P V (V stored transposed)
    (5, 70, 33, 37, False),        # nothing aligned: byte-wise loader, strides not multiples of 16
    (7, 40, 96, 48, True),         # one B shared by every problem
    (1, 50, 50, 16, False),
])
@pytest.mark.parametrize("name", ["m7e4_code", "m4e4_rne"])
def test_batched_gemm_equals_one_gemm_per_problem(case, name):
    Z, M, N, K, shared_b = case
    prod, acc = FORMATS[name]
    A = synth.e4m3_encode(synth.gaussian((Z, M, K), 91) * 100.0)
    B = synth.e4m3_encode(synth.gaussian((N, K) if shared_b else (Z, N, K), 92) * 100.0)
    sa = torch.tensor([0.01])
    sb = torch.linspace(0.5, 1.5, N)
    bias = torch.linspace(-1, 1, N)
    for order, chunk in ((CHK, 16), (SEQ, 16)):
        got = lba.lba_gemm_batched(A.to(DEV), B.to(DEV), sa.to(DEV), sb.to(DEV), bias.to(DEV), prod, acc, order,
                                   chunk).cpu().numpy()
        assert got.shape == (Z, M, N)
        for z in range(Z):
            Bz = B if shared_b else B[z]
            want = ref_gemm(A[z], Bz, sa, sb, bias, prod, acc, order, chunk)
            assert_bit_equal(got[z], want, f"{case} {name} problem {z} order {order}")


def test_batched_gemm_argument_checks():
    prod, acc = code_domain_formats(7, 4)
    one = torch.ones(1, device=DEV)
    A = synth.random_codes((3, 8, 16), 1).to(DEV)
    B = synth.random_codes((3, 8, 16), 2).to(DEV)
    assert lba.lba_gemm_batched(A[:0], B[:0], one, one, None, prod, acc).shape == (0, 8, 8)
    lib = lba.load_library()
    import ctypes as C
    pf, af = lba._fmt(prod), lba._fmt(acc)
    out = torch.empty((3, 8, 8), dtype=torch.float32, device=DEV)
    args = lambda sa_, sb_, so_: (C.c_void_p(A.data_ptr()), C.c_void_p(B.data_ptr()), C.c_void_p(one.data_ptr()), 1,
                                  C.c_void_p(one.data_ptr()), 1, None, 3, 8, 8, 16, sa_, sb_, so_, C.byref(pf),
                                  C.byref(af), CHK, 16, C.c_void_p(out.data_ptr()), None)
    assert lib.lba_gemm_batched(*args(128, 128, 64)) == 0
    assert lib.lba_gemm_batched(*args(128, 128, 63)) == -2     # outputs would overlap
    assert lib.lba_gemm_batched(*args(100, 128, 64)) == -2     # A problems would overlap
    assert lib.lba_gemm_batched(*args(0, 0, 64)) == 0          # shared operands are fine
    torch.cuda.synchronize()


def test_random_formats_shapes_orders_and_data_regimes():
    # a seeded sweep over everything at once: shapes with ragged edges, mantissa / exponent / bias choices around
    # the thresholds that switch kernel variants, floor and nearest-even, with and without the underflow branch,
    # every order, chunk lengths that do and do not fit slabs, and input magnitudes from "everything underflows"
    # to "everything saturates".  Cases that either side rejects as not exactly representable are skipped.
    rng = np.random.default_rng(20240114)
    ran = 0
    variants = set()
    for trial in range(120):
        M, N = int(rng.integers(1, 200)), int(rng.integers(1, 150))
        K = int(rng.choice([1, 5, 16, 31, 48, 100, 160, 333]))
        E = int(rng.integers(3, 7))
        Mb = int(rng.choice([2, 3, 4, 6, 7, 8, 10, 12]))
        rounding = int(rng.integers(0, 2))
        flags = int(rng.integers(0, 2))
        b_prod = 2 ** E - 18 + int(rng.integers(-3, 8))
        b_acc = b_prod - int(rng.integers(0, 4))
        Mp = Mb if rng.random() < 0.7 else int(rng.choice([3, 5, 7, 9]))
        prod = LbaFormat(Mp, E, b_prod, rounding, flags)
        acc = LbaFormat(Mb, E, b_acc, rounding, flags)
        order = SEQ if rng.random() < 0.4 else CHK
        chunk = int(rng.choice([16, 16, 32, 7, 48]))
        scale = float(rng.choice([0.02, 1.0, 30.0, 120.0]))
        A = synth.e4m3_encode(synth.gaussian((M, K), 7000 + trial) * scale)
        B = synth.e4m3_encode(synth.gaussian((N, K), 8000 + trial) * scale)
        if rng.random() < 0.3:
            A, B = A & 0x7F, B & 0x7F                      # same-sign products: the sums run into saturation
        sa = torch.tensor([float(rng.uniform(0.5, 2.0))])
        sb = torch.linspace(0.5, 1.5, N)
        try:
            want = ref_gemm(A, B, sa, sb, None, prod, acc, order, chunk)
        except orc.OracleError:
            continue
        try:
            plan = lba.describe_plan(M, N, K, prod, acc, order, chunk)
            got = gpu_gemm(A, B, sa, sb, None, prod, acc, order, chunk)
        except lba.LbaError as e:
            assert e.status == -3                          # format not carried exactly: refused, never approximated
            continue
        assert_bit_equal(got, want, f"trial {trial}: {M}x{N}x{K} {prod} {acc} order {order}/{chunk} scale {scale} [{plan}]")
        variants.add((plan.split("q=")[1].split()[0], plan.split("order=")[1].split()[0]))
        ran += 1
    assert ran >= 60, ran
    assert len(variants) >= 8, variants


def _overflow_case(M, N, K, regime, seed):
    """E4M3 codes whose chains overflow the accumulator in different ways."""
    A = synth.random_codes((M, K), seed)
    B = synth.random_codes((N, K), seed + 1)
    if regime == 0:                      # Gaussian operands: overflow is rare
        A, _, B, _ = synth.gemm_case(M, N, K, config=seed)
    elif regime == 1:                    # positive products only: the sum climbs to R_OF and stays there
        A, B = A & 0x7F, B & 0x7F
    elif regime == 2:                    # positive head, mixed-sign tail: the last overflow lies mid-chain
        head = max(1, (2 * K) // 3)
        A = torch.cat([A[:, :head] & 0x7F, A[:, head:]], dim=1)
        B = torch.cat([B[:, :head] & 0x7F, B[:, head:]], dim=1)
    return A.contiguous(), B.contiguous()


@pytest.mark.parametrize("name", ["m7e4_code", "m7e4_paper", "m4e4", "m10e5", "m4e3_mnist", "mixed", "m7e4_no_uf"])
def test_last_overflow_index_matches_oracle(name):
    # the re-computation pass of the recursive overflow STE (App. D): last step with |Q_prod(xw) + S| >= R_OF
    prod, acc = FORMATS[name]
    seen_hit = seen_mid = False
    for (M, N, K) in ((1, 1, 1), (70, 45, 37), (130, 67, 160), (64, 64, 576), (33, 129, 1000)):
        for regime in (0, 1, 2, 3):
            A, B = _overflow_case(M, N, K, regime, 100 * regime + K)
            got = lba.lba_gemm_last_overflow(A.to(DEV), B.to(DEV), prod, acc).cpu().numpy()
            want = orc.gemm_last_overflow(A.numpy(), B.numpy(), prod.as_tuple(), acc.as_tuple())
            assert got.dtype == np.int32 and got.shape == (M, N)
            bad = np.argwhere(got != want)
            assert bad.size == 0, (f"{name} {M}x{N}x{K} regime {regime}: {len(bad)} differ; first at {bad[0]}: "
                                   f"gpu={got[tuple(bad[0])]} oracle={want[tuple(bad[0])]}")
            seen_hit |= bool((want >= 0).any())
            seen_mid |= bool(((want >= 0) & (want < K - 1)).any())
    # (the 9-bit, 5-exponent accumulator of "mixed" is out of reach of 1000 products: its answer is -1 everywhere)
    assert name == "mixed" or (seen_hit and seen_mid)


def test_last_overflow_index_edge_cases():
    prod, acc = M7E4_PAPER
    # K = 0: no step, no overflow
    got = lba.lba_gemm_last_overflow(torch.empty((5, 0), dtype=torch.uint8, device=DEV),
                                     torch.empty((7, 0), dtype=torch.uint8, device=DEV), prod, acc)
    assert got.shape == (5, 7) and (got == -1).all()
    assert lba.lba_gemm_last_overflow(torch.empty((0, 8), dtype=torch.uint8, device=DEV),
                                      torch.empty((3, 8), dtype=torch.uint8, device=DEV), prod, acc).shape == (0, 3)
    # hand-worked chain: x = w = 4.0 saturates Q_prod at 15.9375; the fifth step is the first to reach 63.75
    for K, want in ((4, -1), (5, 4), (7, 6), (16, 15), (17, 16)):
        x = torch.full((1, K), 0x48, dtype=torch.uint8, device=DEV)
        assert int(lba.lba_gemm_last_overflow(x, x, prod, acc)[0, 0]) == want
    # odd base pointers go through the byte-wise loader
    Abig = (synth.random_codes((40 * 64 + 3,), 3) & 0x7F).to(DEV)
    Bbig = (synth.random_codes((33 * 64 + 5,), 4) & 0x7F).to(DEV)
    A, B = Abig[3:].view(40, 64), Bbig[5:].view(33, 64)
    got = lba.lba_gemm_last_overflow(A, B, prod, acc).cpu().numpy()
    want = orc.gemm_last_overflow(A.cpu().numpy(), B.cpu().numpy(), prod.as_tuple(), acc.as_tuple())
    assert (got == want).all() and (want >= 0).any()
    # nearest-even quantisers are not covered by this entry point
    with pytest.raises(lba.LbaError):
        lba.lba_gemm_last_overflow(A, B, *FORMATS["m7e4_code_rne"])
    # a NaN code is reported by the dedicated counter, not here; results for finite inputs never depend on it


STE_ORDERS = [(SEQ, 1), (CHK, 16), (CHK, 32), (CHK, 5), (CHK, 4096)]


def _u32(t):
    return t.cpu().numpy().view(np.uint32)


@pytest.mark.parametrize("name", ["m7e4_code", "m7e4_paper", "m4e4", "m10e5", "m4e3_mnist", "m7e4_no_uf"])
@pytest.mark.parametrize("ste", ["of", "diff"])
def test_ste_masks_match_oracle(name, ste):
    # one bit per FMAq step (App. D): first hierarchy and, in chunked order, the folds of the chunk sums
    prod, acc = FORMATS[name]
    kind, e1, e2 = (lba.STE_OF, 0.0, 0.0) if ste == "of" else (lba.STE_DIFF, 2.0 ** -20, 0.25)
    zeros = ones = zeros2 = 0
    for (M, N, K) in ((1, 1, 1), (70, 45, 37), (66, 67, 160), (33, 129, 1000), (130, 68, 1120)):
        for regime in (0, 1, 2, 3):
            A, B = _overflow_case(M, N, K, regime, 100 * regime + K + 7)
            for order, chunk in STE_ORDERS:
                w1, w2 = orc.gemm_ste_mask(A.numpy(), B.numpy(), prod.as_tuple(), acc.as_tuple(), order, chunk,
                                           orc.STE_OF if ste == "of" else orc.STE_DIFF, e1, e2)
                # the overflow masks in sequential and chunk-16 order come from the packed kernel by default and
                # from the scalar tracking kernel under tile override 3: both must give the oracle's bits
                both = ste == "of" and (order == SEQ or chunk == 16)
                for override in ((-1, 3) if both else (-1,)):
                    lba.set_tile_override(override)
                    try:
                        g1, g2 = lba.lba_gemm_ste_mask(A.to(DEV), B.to(DEV), prod, acc, order, chunk, kind, e1, e2)
                    finally:
                        lba.set_tile_override(-1)
                    what = f"{name} {ste} {M}x{N}x{K} regime {regime} order {order} chunk {chunk} override {override}"
                    bad = np.argwhere(_u32(g1) != w1)
                    assert bad.size == 0, f"{what}: mask1 differs in {len(bad)} words, first at {bad[0]}"
                    assert (g2 is None) == (w2 is None)
                    if w2 is not None:
                        bad = np.argwhere(_u32(g2) != w2)
                        assert bad.size == 0, f"{what}: mask2 differs in {len(bad)} words, first at {bad[0]}"
                if w2 is not None:
                    zeros2 += int(w2.size * 32 - np.unpackbits(w2.view(np.uint8)).sum())
                n1 = int(np.unpackbits(w1.view(np.uint8)).sum())
                ones += n1
                zeros += M * N * K - n1
    assert ones > 10000 and zeros > 10000 and zeros2 > 0


def test_ste_mask_edge_cases():
    prod, acc = M7E4_PAPER
    x = torch.full((1, 7), 0x48, dtype=torch.uint8, device=DEV)
    m1, m2 = lba.lba_gemm_ste_mask(x, x, prod, acc, SEQ, 1, lba.STE_OF)
    assert m2 is None and int(m1[0, 0, 0]) == 0b0001111            # hand-worked: four steps stay below 63.75
    m1, m2 = lba.lba_gemm_ste_mask(x, x, prod, acc, CHK, 16, lba.STE_OF)
    assert int(m1[0, 0, 0]) == 0b0001111 and int(m2[0, 0, 0]) == 0  # the one chunk's fold sees 63.75 = R_OF
    # stagnation at 32: the difference estimator stops passing once the product is swamped
    a = torch.full((1, 300), 0x30, dtype=torch.uint8, device=DEV)
    w = torch.full((1, 300), 0x28, dtype=torch.uint8, device=DEV)
    m1, _ = lba.lba_gemm_ste_mask(a, w, prod, acc, SEQ, 1, lba.STE_DIFF, 1e-6, 0.5)
    assert [int(v) & 0xFFFFFFFF for v in m1[0, :, 0]] == [0xFFFFFFFF] * 8 + [0, 0]
    # empty problems, K = 0
    e1, e2 = lba.lba_gemm_ste_mask(torch.empty((3, 0), dtype=torch.uint8, device=DEV),
                                   torch.empty((2, 0), dtype=torch.uint8, device=DEV), prod, acc, CHK, 16, lba.STE_OF)
    assert e1.shape == (3, 0, 2) and e2.shape == (3, 0, 2)
    # odd base pointers: byte-wise loader
    Abig = (synth.random_codes((40 * 64 + 3,), 3) & 0x7F).to(DEV)
    Bbig = (synth.random_codes((33 * 64 + 5,), 4) & 0x7F).to(DEV)
    A, B = Abig[3:].view(40, 64), Bbig[5:].view(33, 64)
    g1, g2 = lba.lba_gemm_ste_mask(A, B, prod, acc, CHK, 16, lba.STE_DIFF, 1e-4, 0.5)
    w1, w2 = orc.gemm_ste_mask(A.cpu().numpy(), B.cpu().numpy(), prod.as_tuple(), acc.as_tuple(), CHK, 16,
                               orc.STE_DIFF, 1e-4, 0.5)
    assert (_u32(g1) == w1).all() and (_u32(g2) == w2).all()
    # rejected arguments
    with pytest.raises(lba.LbaError):
        lba.lba_gemm_ste_mask(A, B, *FORMATS["m7e4_code_rne"], CHK, 16, lba.STE_OF)
    with pytest.raises(lba.LbaError):
        lba.lba_gemm_ste_mask(A, B, prod, acc, CHK, 16, 7)
    with pytest.raises(lba.LbaError):
        lba.lba_gemm_ste_mask(A, B, prod, acc, CHK, 16, lba.STE_DIFF, 0.0, 0.5)
    with pytest.raises(lba.LbaError):
        lba.lba_gemm_ste_mask(A, B, prod, acc, CHK, 16, lba.STE_DIFF, 1e-45, 0.5)


FIXED = {
    "b12_int": (fixed_point_format(16, 0), fixed_point_format(12, 0)),                # integer accumulator, saturating
    "b12_int_wrap": (fixed_point_format(12, 0, True), fixed_point_format(12, 0, True)),
    "finer_product": (fixed_point_format(20, 6), fixed_point_format(16, 2)),         # product re-cut on the coarser grid
    "coarser_product": (fixed_point_format(10, -2), fixed_point_format(14, 3)),
    "b24": (fixed_point_format(24, 5), fixed_point_format(24, 4)),
    "b8_wrap_acc": (fixed_point_format(16, 2), fixed_point_format(8, 1, True)),
    "tiny": (fixed_point_format(2, 0), fixed_point_format(3, -1)),
}


@pytest.mark.parametrize("name", list(FIXED))
def test_fixed_point_accumulators_match_oracle(name):
    # Eq. 1: integer inner loop on the GPU against the exact oracle, every order, ragged shapes, three data regimes
    prod, acc = FIXED[name]
    for (M, N, K) in ((1, 1, 1), (70, 45, 37), (66, 67, 160), (33, 129, 500)):
        for regime in (0, 1, 2):
            if regime == 0:
                A, sa, B, sb = synth.gemm_case(M, N, K, config=40 + K)
            elif regime == 1:
                A, B = synth.random_codes((M, K), 7 + K), synth.random_codes((N, K), 8 + K)
                sa, sb = torch.tensor([0.37]), torch.rand(N, generator=torch.Generator().manual_seed(K)) + 0.5
            else:
                A, B = synth.small_integer_codes((M, K), 9 + K, 15), synth.small_integer_codes((N, K), 10 + K, 15)
                sa, sb = torch.ones(1), torch.ones(1)
            bias = torch.randn(N, generator=torch.Generator().manual_seed(3 * K)) if regime == 1 else None
            for order, chunk in STE_ORDERS:
                got = gpu_gemm(A, B, sa, sb, bias, prod, acc, order, chunk)
                want = ref_gemm(A, B, sa, sb, bias, prod, acc, order, chunk)
                assert_bit_equal(got, want, f"{name} {M}x{N}x{K} regime {regime} order {order} chunk {chunk}")


def test_fixed_point_conv_batched_and_errors():
    prod, acc = FIXED["finer_product"]
    for case in CONV_CASES[:4]:
        b, h, w, cin, cout, kh, kw, stride, pad = case
        x = synth.random_codes((b, h, w, cin), 31)
        wt = synth.random_codes((cout, kh, kw, cin), 32)
        one = torch.ones(1)
        got = lba.lba_conv2d(x.to(DEV), wt.to(DEV), one.to(DEV), one.to(DEV), None, stride, pad, prod, acc, CHK, 16)
        want = orc.conv2d(x.numpy(), wt.numpy(), 1.0, 1.0, None, stride, pad, prod.as_tuple(), acc.as_tuple(), CHK, 16)
        assert_bit_equal(got, want, f"fixed-point conv {case}")
    A = synth.random_codes((3, 20, 48), 41).to(DEV)
    B = synth.random_codes((3, 30, 48), 42).to(DEV)
    one = torch.ones(1, device=DEV)
    got = lba.lba_gemm_batched(A, B, one, one, None, prod, acc, SEQ, 1)
    for z in range(3):
        want = orc.gemm(A[z].cpu().numpy(), B[z].cpu().numpy(), 1.0, 1.0, None, prod.as_tuple(), acc.as_tuple(), SEQ, 1)
        assert_bit_equal(got[z], want, f"fixed-point batched problem {z}")
    assert "q=fixed" in lba.describe_plan(64, 64, 64, prod, acc, CHK, 16)
    a2, b2 = A[0], B[0]
    for bad in ((prod, M7E4_PAPER[1]), (M7E4_PAPER[0], acc), (fixed_point_format(25, 0), acc),
                (LbaFormat(12, 0, 0, 1, 0), acc), (fixed_point_format(16, 13), acc),
                (fixed_point_format(24, 0), fixed_point_format(24, 8))):
        with pytest.raises(lba.LbaError):
            lba.lba_gemm(a2, b2, one, one, None, bad[0], bad[1], SEQ, 1)
    with pytest.raises(lba.LbaError):
        lba.lba_gemm_ste_mask(a2, b2, prod, acc, SEQ, 1, lba.STE_OF)


@pytest.mark.parametrize("name", ["m7e4_code", "m7e4_paper", "m4e4", "m10e5", "mixed", "m4e3_mnist", "m7e4_no_uf"])
def test_cluster_pair_tile_is_exact(name):
    # two CTAs per output tile, each taking every second chunk of 16 (tile override 5): same bits as the oracle
    prod, acc = FORMATS[name]
    lba.set_tile_override(5)
    try:
        assert "pair" in lba.describe_plan(256, 256, 256, prod, acc, CHK, 16)
        for (M, N, K) in ((1, 1, 16), (70, 45, 32), (66, 67, 160), (33, 129, 1008), (130, 68, 1120), (64, 64, 48)):
            for regime in (0, 1, 2, 3):
                A, B = _overflow_case(M, N, K, regime, 50 * regime + K + 3)
                sa = torch.tensor([0.5])
                sb = torch.rand(N, generator=torch.Generator().manual_seed(K)) + 0.5
                got = gpu_gemm(A, B, sa, sb, None, prod, acc, CHK, 16)
                want = ref_gemm(A, B, sa, sb, None, prod, acc, CHK, 16)
                assert_bit_equal(got, want, f"pair tile {name} {M}x{N}x{K} regime {regime}")
        # convolutions with 16-byte taps
        for case in [c for c in CONV_CASES if c[3] % 16 == 0]:
            b, h, w, cin, cout, kh, kw, stride, pad = case
            x = synth.random_codes((b, h, w, cin), 61) & 0x7F
            wt = synth.random_codes((cout, kh, kw, cin), 62)
            one = torch.ones(1)
            got = lba.lba_conv2d(x.to(DEV), wt.to(DEV), one.to(DEV), one.to(DEV), None, stride, pad, prod, acc, CHK, 16)
            want = orc.conv2d(x.numpy(), wt.numpy(), 1.0, 1.0, None, stride, pad, prod.as_tuple(), acc.as_tuple(), CHK, 16)
            assert_bit_equal(got, want, f"pair tile {name} conv {case}")
        # batched problems (the grid's third dimension), per-row scales and a bias; K = 0
        Ab = synth.random_codes((3, 70, 96), 71).to(DEV)
        Bb = synth.random_codes((3, 45, 96), 72).to(DEV)
        sa_rows = (torch.rand(70, generator=torch.Generator().manual_seed(1)) + 0.5).to(DEV)
        sb_cols = (torch.rand(45, generator=torch.Generator().manual_seed(2)) + 0.5).to(DEV)
        bias = torch.randn(45, generator=torch.Generator().manual_seed(3)).to(DEV)
        gb = lba.lba_gemm_batched(Ab, Bb, sa_rows, sb_cols, bias, prod, acc, CHK, 16)
        for z in range(3):
            want = orc.gemm(Ab[z].cpu().numpy(), Bb[z].cpu().numpy(), sa_rows.cpu().numpy(), sb_cols.cpu().numpy(),
                            bias.cpu().numpy(), prod.as_tuple(), acc.as_tuple(), CHK, 16)
            assert_bit_equal(gb[z], want, f"pair tile {name} batched problem {z}")
        empty = lba.lba_gemm(torch.empty((5, 0), dtype=torch.uint8, device=DEV), torch.empty((7, 0), dtype=torch.uint8, device=DEV),
                             torch.ones(1, device=DEV), torch.ones(1, device=DEV), None, prod, acc, CHK, 16)
        assert empty.shape == (5, 7) and (empty == 0).all()
        # not eligible (nearest-even): falls back to the automatic choice, still exact
        pr, ar = FORMATS["m7e4_code_rne"]
        A, B = _overflow_case(40, 40, 64, 3, 5)
        one = torch.ones(1)
        assert "pair" not in lba.describe_plan(40, 40, 64, pr, ar, CHK, 16)
        assert_bit_equal(gpu_gemm(A, B, one, one, None, pr, ar, CHK, 16), ref_gemm(A, B, one, one, None, pr, ar, CHK, 16))
    finally:
        lba.set_tile_override(-1)


def test_random_shapes_pair_tile_masks_and_fixed_point():
    # seeded random shapes, data regimes and formats through the cluster-pair tile, both mask kernels and the
    # fixed-point kernel: every output bit against the oracle
    rng = np.random.default_rng(2024)
    floats = [FORMATS[n] for n in ("m7e4_code", "m7e4_paper", "m4e4", "m10e5", "m4e3_mnist", "m7e4_no_uf", "m5e6")]
    for it in range(48):
        M, N = int(rng.integers(1, 200)), int(rng.integers(1, 200))
        K = int(rng.integers(1, 40)) * 16 if it % 3 else int(rng.integers(1, 700))
        regime = int(rng.integers(0, 3))
        if regime == 2:
            A, _, B, _ = synth.gemm_case(M, N, K, config=300 + it)
        else:
            A, B = synth.random_codes((M, K), 1000 + it), synth.random_codes((N, K), 5000 + it)
            if regime == 1:
                A, B = A & 0x7F, B & 0x7F
        pf, af = floats[it % len(floats)]
        sa, sb = torch.tensor([0.7]), torch.rand(N, generator=torch.Generator().manual_seed(it)) + 0.5
        what = f"case {it}: {M}x{N}x{K} regime {regime}"
        lba.set_tile_override(5)
        try:
            got = gpu_gemm(A, B, sa, sb, None, pf, af, CHK, 16)
        finally:
            lba.set_tile_override(-1)
        assert_bit_equal(got, ref_gemm(A, B, sa, sb, None, pf, af, CHK, 16), what + " pair tile")
        for order, chunk in ((SEQ, 1), (CHK, 16)):
            kinds = [(lba.STE_OF, orc.STE_OF, 0.0, 0.0)] + ([(lba.STE_DIFF, orc.STE_DIFF, 2.0 ** -18, 0.3)] if it % 2 == 0 else [])
            for kind, okind, e1, e2 in kinds:
                g1, g2 = lba.lba_gemm_ste_mask(A.to(DEV), B.to(DEV), pf, af, order, chunk, kind, e1, e2)
                w1, w2 = orc.gemm_ste_mask(A.numpy(), B.numpy(), pf.as_tuple(), af.as_tuple(), order, chunk, okind, e1, e2)
                assert (_u32(g1) == w1).all(), what + f" mask1 order {order} kind {kind}"
                assert w2 is None or (_u32(g2) == w2).all(), what + f" mask2 order {order} kind {kind}"
        bp, ba = int(rng.integers(-8, 8)), int(rng.integers(-10, 8))
        Bp, Ba = int(rng.integers(6, 25)), int(rng.integers(6, 25))
        if ba - bp > 0 and (Bp - 1) + (ba - bp) > 30:
            continue
        fp, fa = fixed_point_format(Bp, bp, bool(it % 2)), fixed_point_format(Ba, ba, bool(it % 2))
        order, chunk = [(SEQ, 1), (CHK, 16), (CHK, 7), (CHK, 48)][it % 4]
        assert_bit_equal(gpu_gemm(A, B, sa, sb, None, fp, fa, order, chunk), ref_gemm(A, B, sa, sb, None, fp, fa, order, chunk),
                         what + f" fixed point {fp.as_tuple()} {fa.as_tuple()} order {order} chunk {chunk}")


M4E3_FORMATS = {
    "m7e4": m4e3_input_formats(7, 4),                                          # the paper's FP8 runs: Q_prod cuts 10 -> 8 bits
    "m7e4_rne": m4e3_input_formats(7, 4, rounding=1),
    "m4e3_acc": (LbaFormat(4, 3, -8, 0, 1 | FLAG_INPUT_M4E3), LbaFormat(4, 3, -10)),   # narrow accumulator: saturates
    "m10e5": m4e3_input_formats(10, 5),                                        # M_prod >= 9: products pass uncut
    "m7e4_flush": (LbaFormat(7, 4, -3, 0, 1 | FLAG_INPUT_M4E3), LbaFormat(7, 4, -5)),  # R_UF_prod = 8: the product flush acts
    "m7e4_sat": (LbaFormat(7, 4, 3, 0, 1 | FLAG_INPUT_M4E3), LbaFormat(7, 4, 1)),      # R_OF_prod = 8160: Q_prod saturates
    "m5e4_rne_no_uf": m4e3_input_formats(5, 4, rounding=1, flags=0),
    "m9e5_rne": m4e3_input_formats(9, 5, rounding=1),
    "wide_rne": (LbaFormat(23, 8, 127, 1, 1 | FLAG_INPUT_M4E3), LbaFormat(23, 8, 127, 1)),
}


@pytest.mark.parametrize("name", list(M4E3_FORMATS))
def test_m4e3_inputs_all_code_pairs_k1(name):
    # the paper's own W/A byte format (Sec. 3.1): every one of the 256 x 256 code pairs through one FMAq
    prod, acc = M4E3_FORMATS[name]
    codes = torch.arange(256, dtype=torch.uint8)[:, None].contiguous()
    one = torch.ones(1)
    got = gpu_gemm(codes, codes, one, one, None, prod, acc, SEQ, 16)
    want = ref_gemm(codes, codes, one, one, None, prod, acc, SEQ, 16)
    assert_bit_equal(got, want, name)
    if name == "m7e4":      # not vacuous: the mantissa cut of Q_prod changed some products
        exact = synth.m4e3_decode(codes).double() @ synth.m4e3_decode(codes).double().T
        assert (torch.from_numpy(want).double() != exact).any()


@pytest.mark.parametrize("name", list(M4E3_FORMATS))
@pytest.mark.parametrize("K", [3, 16, 47, 200, 1024])
def test_m4e3_inputs_random_chains(name, K):
    prod, acc = M4E3_FORMATS[name]
    g = torch.Generator().manual_seed(900 + K)
    A = torch.randint(0, 256, (150, K), generator=g, dtype=torch.uint8)
    B = torch.randint(0, 256, (70, K), generator=g, dtype=torch.uint8)
    sa = torch.tensor([2.0 ** -5])                       # the flex-bias of Sec. 3.1 is the per-tensor power-of-two scale
    sb = torch.tensor([2.0 ** -7])
    for order, chunk in ((SEQ, 16), (CHK, 16), (CHK, 32), (CHK, 5)):
        got = gpu_gemm(A, B, sa, sb, None, prod, acc, order, chunk)
        assert_bit_equal(got, ref_gemm(A, B, sa, sb, None, prod, acc, order, chunk), f"{name} K={K} {order}/{chunk}")


@pytest.mark.parametrize("tile", [0, 1, 2, 3, 5])
def test_m4e3_inputs_every_tile_gaussian_data(tile):
    # Gaussian tensors quantised with a per-tensor flex-bias, ragged shapes, every CTA tile and the byte-wise loader
    for name in ("m7e4", "m7e4_rne"):
        prod, acc = M4E3_FORMATS[name]
        for (M, N, K) in ((200, 100, 576), (129, 65, 147)):
            a, sa = synth.quantise_m4e3_per_tensor(synth.gaussian((M, K), 1100 + M))
            b, sb = synth.quantise_m4e3_per_tensor(synth.gaussian((N, K), 1200 + N, std=0.05))
            lba.set_tile_override(tile)
            try:
                for order in (SEQ, CHK):
                    got = gpu_gemm(a, b, sa, sb, None, prod, acc, order, 16)
                    assert_bit_equal(got, ref_gemm(a, b, sa, sb, None, prod, acc, order, 16), f"{name} tile {tile} {M}x{N}x{K}")
            finally:
                lba.set_tile_override(-1)


def test_m4e3_inputs_convolution_batched_and_rejections():
    prod, acc = M4E3_FORMATS["m7e4"]
    for case in CONV_CASES:
        b, h, w, cin, cout, kh, kw, stride, pad = case
        g = torch.Generator().manual_seed(77)
        x = torch.randint(0, 256, (b, h, w, cin), generator=g, dtype=torch.uint8)
        wt = torch.randint(0, 256, (cout, kh, kw, cin), generator=g, dtype=torch.uint8)
        one = torch.ones(1)
        got = lba.lba_conv2d(x.to(DEV), wt.to(DEV), one.to(DEV), one.to(DEV), None, stride, pad, prod, acc, CHK, 16)
        want = orc.conv2d(x.numpy(), wt.numpy(), 1.0, 1.0, None, stride, pad, prod.as_tuple(), acc.as_tuple(), CHK, 16)
        assert_bit_equal(got, want, f"m4e3 conv {case}")
    A = torch.randint(0, 256, (3, 20, 48), dtype=torch.uint8, generator=torch.Generator().manual_seed(5)).to(DEV)
    B = torch.randint(0, 256, (3, 30, 48), dtype=torch.uint8, generator=torch.Generator().manual_seed(6)).to(DEV)
    one = torch.ones(1, device=DEV)
    got = lba.lba_gemm_batched(A, B, one, one, None, prod, acc, CHK, 16)
    for z in range(3):
        assert_bit_equal(got[z], orc.gemm(A[z].cpu().numpy(), B[z].cpu().numpy(), 1.0, 1.0, None, prod.as_tuple(),
                                          acc.as_tuple(), CHK, 16), f"m4e3 batched {z}")
    # the fixed-point accumulators and the straight-through-estimator passes take E4M3 operands only
    fx = LbaFormat(12, 0, -7, 0, FLAG_INPUT_M4E3)
    with pytest.raises(lba.LbaError) as e:
        lba.lba_gemm(A[0], B[0], one, one, None, fx, fixed_point_format(12, -9), SEQ, 1)
    assert e.value.status == -3
    with pytest.raises(lba.LbaError) as e:
        lba.lba_gemm_ste_mask(A[0], B[0], prod, acc, CHK, 16, lba.STE_OF)
    assert e.value.status == -3
    with pytest.raises(lba.LbaError) as e:
        lba.lba_gemm_last_overflow(A[0], B[0], prod, acc)
    assert e.value.status == -3


def test_zero_and_empty_shapes():
    prod, acc = code_domain_formats(7, 4)
    one = torch.ones(1)
    A = synth.random_codes((5, 0), 1)
    B = synth.random_codes((7, 0), 2)
    got = gpu_gemm(A, B, one, one, torch.arange(7, dtype=torch.float32), prod, acc, CHK, 16).cpu().numpy()
    assert got.shape == (5, 7) and np.array_equal(got, np.tile(np.arange(7, dtype=np.float32), (5, 1)))
    assert gpu_gemm(synth.random_codes((0, 8), 1), synth.random_codes((3, 8), 2), one, one, None, prod, acc, CHK,
                    16).shape == (0, 3)
    # negative-zero inputs and exact cancellation give +0
    A = torch.tensor([[0x80, 0x38, 0xB8, 0x00]], dtype=torch.uint8)       # -0, 1, -1, 0
    B = torch.tensor([[0x38, 0x40, 0x40, 0x38]], dtype=torch.uint8)       # 1, 2, 2, 1
    for fmts in ((WIDE, WIDE), FORMATS["wide_rne"], code_domain_formats(7, 4, flags=0)):
        got = gpu_gemm(A, B, one, one, None, *fmts, SEQ, 16).cpu().numpy()
        assert got[0, 0] == 0 and not np.signbit(got[0, 0])


def test_unaligned_operands_take_the_bytewise_loader():
    prod, acc = code_domain_formats(7, 4)
    one = torch.ones(1, device=DEV)
    Abig = synth.random_codes((40 * 64 + 3,), 3).to(DEV)
    Bbig = synth.random_codes((33 * 64 + 5,), 4).to(DEV)
    A = Abig[3:].view(40, 64)          # K % 16 == 0 but the base pointer is odd
    B = Bbig[5:].view(33, 64)
    assert A.data_ptr() % 16 != 0
    got = lba.lba_gemm(A, B, one, one, None, prod, acc, CHK, 16)
    want = orc.gemm(A.cpu().numpy(), B.cpu().numpy(), 1.0, 1.0, None, prod.as_tuple(), acc.as_tuple(), CHK, 16)
    assert_bit_equal(got, want)


CONV_CASES = [
    # B, H, W, Cin, Cout, KH, KW, stride, pad
    (2, 12, 12, 3, 64, 7, 7, (2, 2), (3, 3)),      # stem-like: C_in = 3, K = 147, byte-wise loader
    (2, 9, 9, 16, 40, 3, 3, (1, 1), (1, 1)),       # vector loader, padding on all sides
    (1, 14, 14, 64, 130, 3, 3, (2, 2), (1, 1)),    # stride 2
    (3, 8, 8, 32, 70, 1, 1, (2, 2), (0, 0)),       # 1x1 downsample
    (1, 7, 9, 5, 3, 3, 2, (2, 1), (0, 2)),         # odd everything
    (1, 5, 5, 48, 33, 5, 5, (1, 1), (2, 2)),
]


@pytest.mark.parametrize("case", CONV_CASES)
@pytest.mark.parametrize("name", ["m7e4_code", "m7e4_paper", "m4e4_rne", "m10e5", "m10e6_rne"])
def test_conv2d_matches_direct_convolution(case, name):
    # (the padded cases also hold slabs in which every row of a tile is zero while some outputs sit at R_OF and
    # others, past the edge of the matrix, are zero: the clamp bookkeeping must take the same path in every lane)
    B, H, W, Cin, Cout, KH, KW, stride, pad = case
    prod, acc = FORMATS[name]
    x = synth.random_codes((B, H, W, Cin), 30)
    w = synth.random_codes((Cout, KH, KW, Cin), 31)
    sx = torch.tensor([0.37])
    sw = torch.linspace(0.5, 2.0, Cout)
    bias = torch.linspace(-3, 3, Cout)
    for order, chunk in ((SEQ, 16), (CHK, 16), (CHK, 7)):
        got = lba.lba_conv2d(x.to(DEV), w.to(DEV), sx.to(DEV), sw.to(DEV), bias.to(DEV), stride, pad, prod, acc,
                             order, chunk)
        want = orc.conv2d(x.numpy(), w.numpy(), sx.numpy(), sw.numpy(), bias.numpy(), stride, pad, prod.as_tuple(),
                          acc.as_tuple(), order, chunk)
        assert tuple(got.shape) == want.shape
        assert_bit_equal(got, want, f"{case} {name} {order}/{chunk}")


def test_random_convolution_geometries():
    rng = np.random.default_rng(424242)
    for trial in range(40):
        B, H, W = int(rng.integers(1, 4)), int(rng.integers(3, 20)), int(rng.integers(3, 20))
        Cin = int(rng.choice([1, 3, 5, 16, 24, 32, 48]))
        Cout = int(rng.integers(1, 90))
        KH, KW = int(rng.integers(1, 6)), int(rng.integers(1, 6))
        stride = (int(rng.integers(1, 4)), int(rng.integers(1, 4)))
        pad = (int(rng.integers(0, 3)), int(rng.integers(0, 3)))
        if H + 2 * pad[0] < KH or W + 2 * pad[1] < KW:
            continue
        name = ["m7e4_code", "m4e4", "m7e4_code_rne"][trial % 3]
        prod, acc = FORMATS[name]
        x = synth.e4m3_encode(synth.gaussian((B, H, W, Cin), 9000 + trial).relu() * 60.0)
        w = synth.e4m3_encode(synth.gaussian((Cout, KH, KW, Cin), 9500 + trial) * 60.0)
        sx = torch.tensor([0.7])
        sw = torch.linspace(0.5, 2.0, Cout)
        order, chunk = [(CHK, 16), (SEQ, 16), (CHK, 32), (CHK, 5)][trial % 4]
        got = lba.lba_conv2d(x.to(DEV), w.to(DEV), sx.to(DEV), sw.to(DEV), None, stride, pad, prod, acc, order, chunk)
        want = orc.conv2d(x.numpy(), w.numpy(), sx.numpy(), sw.numpy(), None, stride, pad, prod.as_tuple(),
                          acc.as_tuple(), order, chunk)
        assert tuple(got.shape) == want.shape
        assert_bit_equal(got, want, f"trial {trial}: B{B} {H}x{W}x{Cin}->{Cout} k{KH}x{KW} s{stride} p{pad} {name} {order}/{chunk}")


@pytest.mark.parametrize("tile", [0, 1, 2, 3])
def test_conv2d_every_tile(tile):
    prod, acc = code_domain_formats(7, 4)
    lba.set_tile_override(tile)
    try:
        for case in CONV_CASES[:3]:
            B, H, W, Cin, Cout, KH, KW, stride, pad = case
            x, sx = synth.quantise_per_tensor(synth.gaussian((B, H, W, Cin), 40).relu())
            w, sw = synth.quantise_per_channel(synth.he_normal((Cout, KH, KW, Cin), KH * KW * Cin, 41))
            got = lba.lba_conv2d(x.to(DEV), w.to(DEV), sx.to(DEV), sw.to(DEV), None, stride, pad, prod, acc, CHK, 16)
            want = orc.conv2d(x.numpy(), w.numpy(), sx.numpy(), sw.numpy(), None, stride, pad, prod.as_tuple(),
                              acc.as_tuple(), CHK, 16)
            assert_bit_equal(got, want, f"tile {tile} {case}")
    finally:
        lba.set_tile_override(-1)


def test_host_buffer_entry_points():
    prod, acc = code_domain_formats(7, 4)
    A, sa, B, sb = synth.gemm_case(200, 96, 128, config=9)
    bias = torch.linspace(-1, 1, 96)
    out = torch.empty((200, 96), dtype=torch.float32).pin_memory()
    ws = torch.empty(lba.gemm_host_workspace_bytes(200, 96, 128, 1, 1, True), dtype=torch.uint8, device=DEV)
    lba.lba_gemm_host(A.pin_memory(), B.pin_memory(), sa, sb, bias, prod, acc, CHK, 16, out, ws)
    torch.cuda.synchronize()
    assert_bit_equal(out, ref_gemm(A, B, sa, sb, bias, prod, acc, CHK, 16))
    B_, H, W, Cin, Cout, KH, KW, stride, pad = CONV_CASES[1]
    x = synth.random_codes((B_, H, W, Cin), 50)
    w = synth.random_codes((Cout, KH, KW, Cin), 51)
    one = torch.ones(1)
    Ho, Wo = lba.conv_out_hw(H, W, KH, KW, stride, pad)
    out = torch.empty((B_, Ho, Wo, Cout), dtype=torch.float32).pin_memory()
    ws = torch.empty(lba.conv2d_host_workspace_bytes(B_, H, W, Cin, Cout, KH, KW, stride, pad, 1, 1, False),
                     dtype=torch.uint8, device=DEV)
    lba.lba_conv2d_host(x, w, one, one, None, stride, pad, prod, acc, CHK, 16, out, ws)
    torch.cuda.synchronize()
    assert_bit_equal(out, orc.conv2d(x.numpy(), w.numpy(), 1.0, 1.0, None, stride, pad, prod.as_tuple(),
                                     acc.as_tuple(), CHK, 16))
    with pytest.raises(lba.LbaError) as e:
        lba.lba_gemm_host(A, B, sa, sb, bias, prod, acc, CHK, 16, torch.empty((200, 96)), ws[:16])
    assert e.value.status == -7


def test_nan_code_counter():
    codes = synth.random_codes((100000,), 60)
    assert lba.count_nan_codes(codes.to(DEV)) == 0
    codes[17] = 0x7F
    codes[99999] = 0xFF
    assert lba.count_nan_codes(codes.to(DEV)) == 2


def test_calls_are_capturable_in_a_cuda_graph():
    # the entry points only enqueue work on the given stream (no allocation, no synchronisation), so a stream capture
    # records them; the replayed graph gives the oracle's bits for GEMM and convolution alike, on fresh operands too
    prod, acc = code_domain_formats(7, 4)
    A, sa, B, sb = synth.gemm_case(70, 45, 100, config=3)
    dA, dB, dsa, dsb = A.to(DEV), B.to(DEV), sa.to(DEV), sb.to(DEV)
    out = torch.zeros((70, 45), dtype=torch.float32, device=DEV)
    x = synth.random_codes((2, 9, 9, 16), 30).to(DEV)
    w = synth.random_codes((40, 3, 3, 16), 31).to(DEV)
    one = torch.ones(1, device=DEV)
    cout = torch.zeros((2, 9, 9, 40), dtype=torch.float32, device=DEV)
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):   # first use outside the capture (function attributes are set once per kernel)
        lba.lba_gemm(dA, dB, dsa, dsb, None, prod, acc, CHK, 16, out=out)
        lba.lba_conv2d(x, w, one, one, None, (1, 1), (1, 1), prod, acc, CHK, 16, out=cout)
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph, stream=side):
        lba.lba_gemm(dA, dB, dsa, dsb, None, prod, acc, CHK, 16, out=out)
        lba.lba_conv2d(x, w, one, one, None, (1, 1), (1, 1), prod, acc, CHK, 16, out=cout)
    torch.cuda.current_stream().wait_stream(side)
    A2 = synth.random_codes((70, 100), 77)
    dA.copy_(A2.to(DEV))
    out.zero_()
    cout.zero_()
    graph.replay()
    torch.cuda.synchronize()
    assert_bit_equal(out, ref_gemm(A2, B, sa, sb, None, prod, acc, CHK, 16), "graph replay, GEMM")
    want = orc.conv2d(x.cpu().numpy(), w.cpu().numpy(), 1.0, 1.0, None, (1, 1), (1, 1), prod.as_tuple(), acc.as_tuple(), CHK, 16)
    assert_bit_equal(cout, want, "graph replay, convolution")
