"""Seeded random differential test of the CUDA path against the CPU oracle, bit for bit: random entry points (GEMM, batched,
host buffers, convolution, fixed point, STE masks, last overflow), formats (M, E, bias, rounding, underflow flag, input byte
format), shapes, orders, chunk sizes, scale layouts, tile shapes and operand distributions.

The number of cases of the default run is small; LBA_FUZZ_CASES, LBA_FUZZ_SEED and LBA_FUZZ_SCALE widen it."""
import os

import numpy as np
import pytest
import torch

from oracle import lba_oracle as orc
from paper_2401_14110_b200 import binding as lba
from paper_2401_14110_b200 import synth
from paper_2401_14110_b200 import LbaFormat, FLAG_INPUT_M4E3, ORDER_SEQUENTIAL as SEQ, ORDER_CHUNKED as CHK

pytestmark = pytest.mark.gpu

DEV = "cuda:0"
CASES = int(os.environ.get("LBA_FUZZ_CASES", "400"))
SEED = int(os.environ.get("LBA_FUZZ_SEED", "20240125"))
SCALE = int(os.environ.get("LBA_FUZZ_SCALE", "1"))   # multiplies the largest M and N drawn (several 128-wide tiles per side)
ERR_FORMAT = -3
UNCHECKED = []   # cases the library ran and the oracle could not carry


def _codes(rng, shape, kind, m4e3):
    """Operand bytes: uniform codes, Gaussian values, one sign only (sums climb to R_OF), or mostly zeros."""
    n = int(np.prod(shape))
    if m4e3:
        c = rng.integers(0, 256, n, dtype=np.uint8)
    else:
        finite = np.array([b for b in range(256) if (b & 0x7F) != 0x7F], dtype=np.uint8)
        c = finite[rng.integers(0, finite.size, n)]
    if kind == "gauss" and not m4e3:
        v = torch.from_numpy(rng.standard_normal(n).astype(np.float32) * float(rng.choice([0.05, 1.0, 30.0, 200.0])))
        c = synth.e4m3_encode(v.clamp(-448, 448)).numpy()
    elif kind == "one_sign":
        c = c & 0x7F
    elif kind == "sparse":
        c = np.where(rng.random(n) < 0.85, 0, c).astype(np.uint8)
    elif kind == "small":
        c = (c & 0x87) | (rng.integers(0, 3, n, dtype=np.uint8) << 3)   # the lowest binades: products near R_UF
    elif kind == "climb":
        c = (c & 0x07) | (rng.integers(3, 9, n, dtype=np.uint8) << 3)   # one sign, middle binades: sums climb slowly to R_OF
    return torch.from_numpy(np.ascontiguousarray(c.reshape(shape)))


def _formats(rng):
    m4e3 = bool(rng.random() < 0.25)
    rounding = int(rng.random() < 0.4)
    flags = int(rng.random() < 0.8)
    if rng.random() < 0.5:       # around the flex-bias rule of Sec. 3.1
        E = int(rng.integers(3, 8))
        M = int(rng.choice([2, 3, 4, 5, 7, 8, 10, 12]))
        bp = 2 ** E - (16 if m4e3 else 18) + int(rng.integers(-3, 4))
        prod = LbaFormat(M, E, bp, rounding, flags | (FLAG_INPUT_M4E3 if m4e3 else 0))
        acc = LbaFormat(int(rng.choice([M, M, max(1, M - 2), min(23, M + 3)])), E, bp - int(rng.integers(0, 5)), rounding, flags)
    else:                        # anything the header admits (the far ends of the bias range now and then)
        lo, hi = (-96, 193) if rng.random() < 0.2 else (-20, 40)
        prod = LbaFormat(int(rng.integers(1, 24)), int(rng.integers(1, 9)), int(rng.integers(lo, hi)), rounding,
                         flags | (FLAG_INPUT_M4E3 if m4e3 else 0))
        acc = LbaFormat(int(rng.integers(1, 24)), int(rng.integers(1, 9)), int(rng.integers(lo, hi)), rounding, flags)
    return prod, acc, m4e3


def _fixed_formats(rng):
    """Q^FIXED of Eq. 1 for product and accumulator: B bits with the sign, step 2^-b, saturating or wrapping."""
    bp, ba = int(rng.integers(-6, 9)), int(rng.integers(-6, 9))
    wrap = int(rng.random() < 0.3) * 2
    return (LbaFormat(int(rng.integers(2, 25)), 0, bp, 0, wrap if rng.random() < 0.5 else 0),
            LbaFormat(int(rng.integers(2, 25)), 0, ba, 0, wrap), False)


def _differ(got, want, what):
    g = np.ascontiguousarray(got).view(np.uint32).reshape(-1)
    w = np.ascontiguousarray(want, dtype=got.dtype).view(np.uint32).reshape(-1)
    assert g.shape == w.shape, f"{what}: shapes {got.shape} and {np.shape(want)}"
    bad = np.nonzero(g != w)[0]
    assert bad.size == 0, (f"{what}: {bad.size} of {g.size} outputs differ; first at {bad[0]}: gpu={got.reshape(-1)[bad[0]]!r} "
                           f"oracle={np.asarray(want).reshape(-1)[bad[0]]!r}")


def _one_case(rng, trial):
    kind = str(rng.choice(["gemm"] * 10 + ["conv"] * 3 + ["fixed"] * 2 + ["batched", "host", "static", "ste", "ste", "last"]))
    prod, acc, m4e3 = _fixed_formats(rng) if kind == "fixed" else _formats(rng)
    if kind in ("ste", "last"):     # floor rounding and E4M3 bytes only
        prod = LbaFormat(prod.man_bits, prod.exp_bits, prod.bias, 0, prod.flags & 1)
        acc = LbaFormat(acc.man_bits, acc.exp_bits, acc.bias, 0, acc.flags & 1)
        m4e3 = False
    small = kind in ("ste", "last", "conv")
    M, N = int(rng.integers(1, (120 if small else 280) * SCALE)), int(rng.integers(1, (120 if small else 280) * SCALE))
    K = int(rng.choice([0, 1, 2, 15, 16, 17, 31, 33, 64, 100, 255, 256, 500, int(rng.integers(1, 700)), int(rng.integers(1, 700))]))
    if kind in ("gemm", "fixed", "host") and rng.random() < 0.03:     # a few long chains and wide shapes
        K = int(rng.choice([1000, 2048, 4100]))
        M, N = (int(rng.integers(1, 700)), int(rng.integers(1, 130))) if rng.random() < 0.5 else (M, N)
    order = SEQ if (rng.random() < 0.35 or kind == "last") else CHK
    chunk = int(rng.choice([16, 16, 16, 1, 2, 7, 32, 48, 64, int(rng.integers(1, 100))]))
    tile = int(rng.choice([-1, -1, -1, 0, 1, 2, 3, 5]))
    ka, kb = rng.choice(["uniform", "gauss", "one_sign", "sparse", "small", "climb"], 2)
    stride = pad = None
    misaligned = bool(rng.random() < 0.15)
    if kind == "conv":
        Bn, H, W = int(rng.integers(1, 4)), int(rng.integers(1, 16)), int(rng.integers(1, 16))
        Cin = int(rng.choice([1, 3, 4, 5, 16, 24, 32, 48, 64]))
        KH, KW = int(rng.integers(1, 6)), int(rng.integers(1, 6))
        stride = (int(rng.integers(1, 4)), int(rng.integers(1, 4)))
        pad = (int(rng.integers(0, 4)), int(rng.integers(0, 4)))
        if min(orc.conv_out_hw(H, W, KH, KW, stride, pad)) < 1:
            return False
        A, B = _codes(rng, (Bn, H, W, Cin), ka, m4e3), _codes(rng, (N, KH, KW, Cin), kb, m4e3)
        M, K = Bn, KH * KW * Cin
        sa = torch.from_numpy(rng.uniform(0.25, 4.0, 1).astype(np.float32))
    else:
        Z = int(rng.integers(1, 4)) if kind == "batched" else None
        A = _codes(rng, (M, K) if Z is None else (Z, M, K), ka, m4e3)
        B = _codes(rng, (N, K) if (Z is None or rng.random() < 0.4) else (Z, N, K), kb, m4e3)
        sa = torch.from_numpy(rng.uniform(0.25, 4.0, M if rng.random() < 0.5 else 1).astype(np.float32))
    sb = torch.from_numpy(rng.uniform(1e-3, 2.0, N if rng.random() < 0.5 else 1).astype(np.float32))
    bias = torch.from_numpy(rng.standard_normal(N).astype(np.float32)) if rng.random() < 0.5 else None
    ste = (lba.STE_OF, 0.0, 0.0) if rng.random() < 0.5 else (lba.STE_DIFF, float(rng.choice([1e-6, 1e-4, 1e-2])),
                                                             float(rng.choice([0.25, 0.5])))
    what = (f"trial {trial} {kind}: prod={prod.as_tuple()} acc={acc.as_tuple()} A{tuple(A.shape)} B{tuple(B.shape)} order={order} "
            f"chunk={chunk} tile={tile} A={ka} B={kb} sa={sa.numel()} sb={sb.numel()} bias={bias is not None} "
            f"stride={stride} pad={pad} ste={ste}")
    d = lambda t: None if t is None else t.to(DEV)
    n = lambda t: None if t is None else t.numpy()
    pt, at = prod.as_tuple(), acc.as_tuple()
    lba.set_tile_override(tile)
    try:
        if kind == "conv":
            got = lba.lba_conv2d(d(A), d(B), d(sa), d(sb), d(bias), stride, pad, prod, acc, order, chunk)
        elif kind == "batched":
            got = lba.lba_gemm_batched(d(A), d(B), d(sa), d(sb), d(bias), prod, acc, order, chunk)
        elif kind == "host":
            got = torch.empty((M, N), dtype=torch.float32)
            ws = torch.empty(lba.gemm_host_workspace_bytes(M, N, K, sa.numel(), sb.numel(), bias is not None) + 256,
                             dtype=torch.uint8, device=DEV)
            lba.lba_gemm_host(A, B, sa, sb, bias, prod, acc, order, chunk, got, ws)
            torch.cuda.synchronize()
        elif kind == "static":
            got = torch.empty((M, N), dtype=torch.float32)
            lba.lba_gemm_host_static(A, B, sa, sb, bias, prod, acc, order, chunk, got)
            torch.cuda.synchronize()
        elif kind == "ste":
            got = lba.lba_gemm_ste_mask(d(A), d(B), prod, acc, order, chunk, *ste)
        elif kind == "last":
            got = lba.lba_gemm_last_overflow(d(A), d(B), prod, acc)
        else:
            # now and then from operands and into an output that start off a 16-byte boundary (the byte-wise loader, scalar stores)
            shift = lambda t, o: torch.cat([t.new_zeros(o), t.reshape(-1)])[o:].view(t.shape)
            oa, ob, oo = (int(v) for v in rng.integers(0, 16, 3)) if misaligned else (0, 0, 0)
            out = shift(torch.empty((M, N), dtype=torch.float32, device=DEV), oo % 4)
            got = lba.lba_gemm(shift(d(A), oa), shift(d(B), ob), d(sa), d(sb), d(bias), prod, acc, order, chunk, out=out)
    except lba.LbaError as e:
        assert e.status == ERR_FORMAT, what + f": {e}"
        return False
    finally:
        lba.set_tile_override(-1)
    try:
        _compare(kind, got, A, B, sa, sb, bias, stride, pad, pt, at, order, chunk, ste, what)
    except orc.OracleError:   # the span of the operands exceeds the oracle's exact 126-bit carrier: the case cannot be checked
        UNCHECKED.append(what)
        return False
    return True


def _compare(kind, got, A, B, sa, sb, bias, stride, pad, pt, at, order, chunk, ste, what):
    n = lambda t: None if t is None else t.numpy()
    if kind == "conv":
        _differ(got.cpu().numpy(), orc.conv2d(n(A), n(B), n(sa), n(sb), n(bias), stride, pad, pt, at, order, chunk), what)
    elif kind == "batched":
        for z in range(A.shape[0]):
            Bz = B if B.dim() == 2 else B[z]
            _differ(got[z].cpu().numpy(), orc.gemm(n(A[z]), n(Bz), n(sa), n(sb), n(bias), pt, at, order, chunk), what + f" z={z}")
    elif kind == "ste":
        w1, w2 = orc.gemm_ste_mask(n(A), n(B), pt, at, order, chunk, orc.STE_OF if ste[0] == lba.STE_OF else orc.STE_DIFF,
                                   ste[1], ste[2])
        _differ(got[0].cpu().numpy(), w1, what + " mask1")
        assert (got[1] is None) == (w2 is None), what
        if w2 is not None:
            _differ(got[1].cpu().numpy(), w2, what + " mask2")
    elif kind == "last":
        _differ(got.cpu().numpy(), orc.gemm_last_overflow(n(A), n(B), pt, at), what)
    else:
        _differ(got.cpu().numpy(), orc.gemm(n(A), n(B), n(sa), n(sb), n(bias), pt, at, order, chunk), what)


def test_random_formats_shapes_and_operands():
    rng = np.random.default_rng(SEED)
    ran = sum(_one_case(rng, t) for t in range(CASES))
    # formats the library declines (a carrier out of binary32's range, 22 mantissa bits with nearest-even, ...) are
    # declined with the format status; most draws must run
    assert ran >= CASES // 2, f"only {ran} of {CASES} random cases were accepted"
    assert len(UNCHECKED) <= CASES // 50, f"{len(UNCHECKED)} cases could not be checked, e.g. {UNCHECKED[0]}"
