"""ctypes access to the C++ oracle (``lba_oracle.cpp``).  TEST INFRASTRUCTURE ONLY.

Arrays are numpy: uint8 for E4M3 bytes, float32 for scales, bias and outputs.
A format is a tuple ``(M, E, b, rounding, flags)`` as in Eq. 2 of the paper, with
``rounding`` 0 = floor on the magnitude, 1 = nearest-even and ``flags`` bit0 = underflow on;
bit2 on the product format says that the input bytes are codes of the paper's M4E3 W/A format.
"""
import ctypes as C
import os

import numpy as np

from . import build as _build

SEQUENTIAL = 0
CHUNKED = 1

ROUND_FLOOR = 0
ROUND_NEAREST_EVEN = 1
FLAG_UNDERFLOW = 1
FLAG_INPUT_M4E3 = 4


class OracleError(RuntimeError):
    def __init__(self, status):
        names = {-1: "bad argument", -2: "format outside the oracle's domain", -3: "E4M3 NaN code in the input",
                 -4: "value left the exact carrier or the binary32 range"}
        super().__init__(f"oracle status {status}: {names.get(status, 'unknown')}")
        self.status = status


class _Fmt(C.Structure):
    _fields_ = [("man_bits", C.c_int32), ("exp_bits", C.c_int32), ("bias", C.c_int32),
                ("rounding", C.c_int32), ("flags", C.c_int32)]


def _fmt(f):
    M, E, b, rounding, flags = f
    return _Fmt(int(M), int(E), int(b), int(rounding), int(flags))


_lib = None


def lib():
    global _lib
    if _lib is None:
        _lib = C.CDLL(_build.build())
        _lib.lbo_version.restype = C.c_int
    return _lib


def _check(st):
    if st != 0:
        raise OracleError(st)


def _u8(a):
    a = np.ascontiguousarray(a, dtype=np.uint8)
    return a, a.ctypes.data_as(C.POINTER(C.c_uint8))


def _f32(a):
    a = np.ascontiguousarray(np.atleast_1d(a), dtype=np.float32)
    return a, a.ctypes.data_as(C.POINTER(C.c_float))


def _i64(a):
    a = np.ascontiguousarray(a, dtype=np.int64)
    return a, a.ctypes.data_as(C.POINTER(C.c_int64))


def default_threads():
    return len(os.sched_getaffinity(0))


def decode_e4m3(code):
    v = C.c_double()
    _check(lib().lbo_decode_e4m3(C.c_uint8(int(code)), C.byref(v)))
    return v.value


def decode_m4e3(code):
    v = C.c_double()
    _check(lib().lbo_decode_m4e3(C.c_uint8(int(code)), C.byref(v)))
    return v.value


def fmt_range(fmt):
    """(R_OF, R_UF) of Eq. 2."""
    f = _fmt(fmt)
    r_of, r_uf = C.c_double(), C.c_double()
    _check(lib().lbo_range(C.byref(f), C.byref(r_of), C.byref(r_uf)))
    return r_of.value, r_uf.value


def quantise(fmt, x):
    f = _fmt(fmt)
    y = C.c_double()
    _check(lib().lbo_quantise(C.byref(f), C.c_double(float(x)), C.byref(y)))
    return y.value


def dot(prod_fmt, acc_fmt, order, chunk, x, w, trace=False):
    """One output scalar from two byte vectors; optionally the running first-hierarchy sums."""
    x, xp = _u8(x)
    w, wp = _u8(w)
    assert x.ndim == 1 and x.shape == w.shape
    K = x.shape[0]
    pf, af = _fmt(prod_fmt), _fmt(acc_fmt)
    y = C.c_double()
    tr = np.zeros(K, dtype=np.float64) if trace else None
    trp = tr.ctypes.data_as(C.POINTER(C.c_double)) if trace else None
    _check(lib().lbo_dot(C.byref(pf), C.byref(af), C.c_int(order), C.c_int64(chunk), xp, C.c_int64(1), wp,
                         C.c_int64(1), C.c_int64(K), C.byref(y), trp))
    return (y.value, tr) if trace else y.value


def fmaq_grid(prod_fmt, acc_fmt, xcodes, wcodes, s_values, nthreads=0):
    """float64 [len(s_values)][len(xcodes)][len(wcodes)]: one FMAq step (Eq. 4) from every given running sum."""
    x, xp = _u8(xcodes)
    w, wp = _u8(wcodes)
    sv = np.ascontiguousarray(s_values, dtype=np.float64)
    pf, af = _fmt(prod_fmt), _fmt(acc_fmt)
    out = np.empty((sv.size, x.size, w.size), dtype=np.float64)
    _check(lib().lbo_fmaq_grid(C.byref(pf), C.byref(af), xp, C.c_int64(x.size), wp, C.c_int64(w.size),
                               sv.ctypes.data_as(C.POINTER(C.c_double)), C.c_int64(sv.size),
                               out.ctypes.data_as(C.POINTER(C.c_double)), C.c_int(nthreads or default_threads())))
    return out


def _scales(sa, sb, bias, la, lb):
    sa, sap = _f32(sa)
    sb, sbp = _f32(sb)
    assert sa.size in (1, la) and sb.size in (1, lb)
    if bias is not None:
        bias, bp = _f32(bias)
        assert bias.size == lb
    else:
        bp = None
    return (sa, sb, bias), sap, sa.size, sbp, sb.size, bp


def gemm(A, B, scale_a, scale_b, bias, prod_fmt, acc_fmt, order, chunk, nthreads=0):
    """out[M][N] for A [M][K], B [N][K] (bytes)."""
    A, Ap = _u8(A)
    B, Bp = _u8(B)
    M, K = A.shape
    N, K2 = B.shape
    assert K == K2
    keep, sap, sal, sbp, sbl, bp = _scales(scale_a, scale_b, bias, M, N)
    pf, af = _fmt(prod_fmt), _fmt(acc_fmt)
    out = np.empty((M, N), dtype=np.float32)
    _check(lib().lbo_gemm(Ap, Bp, sap, C.c_int(sal), sbp, C.c_int(sbl), bp, C.c_int64(M), C.c_int64(N),
                          C.c_int64(K), C.byref(pf), C.byref(af), C.c_int(order), C.c_int64(chunk),
                          out.ctypes.data_as(C.POINTER(C.c_float)), C.c_int(nthreads or default_threads())))
    return out


def gemm_points(A, B, scale_a, scale_b, bias, prod_fmt, acc_fmt, order, chunk, ms, ns, nthreads=0):
    """Selected elements (ms[p], ns[p]) of the same GEMM."""
    A, Ap = _u8(A)
    B, Bp = _u8(B)
    M, K = A.shape
    N, _ = B.shape
    keep, sap, sal, sbp, sbl, bp = _scales(scale_a, scale_b, bias, M, N)
    pf, af = _fmt(prod_fmt), _fmt(acc_fmt)
    ms, msp = _i64(ms)
    ns, nsp = _i64(ns)
    P = ms.size
    assert ns.size == P
    out = np.empty(P, dtype=np.float32)
    _check(lib().lbo_gemm_points(Ap, Bp, sap, C.c_int(sal), sbp, C.c_int(sbl), bp, C.c_int64(M), C.c_int64(N),
                                 C.c_int64(K), C.byref(pf), C.byref(af), C.c_int(order), C.c_int64(chunk), msp, nsp,
                                 C.c_int64(P), out.ctypes.data_as(C.POINTER(C.c_float)),
                                 C.c_int(nthreads or default_threads())))
    return out


def gemm_last_overflow(A, B, prod_fmt, acc_fmt, nthreads=0):
    """int32 [M][N]: last sequential step at which the input of Q_acc reached R_OF (STE^OF = 0, App. D), -1 if none."""
    A, Ap = _u8(A)
    B, Bp = _u8(B)
    M, K = A.shape
    N, _ = B.shape
    pf, af = _fmt(prod_fmt), _fmt(acc_fmt)
    out = np.empty((M, N), dtype=np.int32)
    _check(lib().lbo_gemm_last_overflow(Ap, Bp, C.c_int64(M), C.c_int64(N), C.c_int64(K), C.byref(pf), C.byref(af),
                                        out.ctypes.data_as(C.POINTER(C.c_int32)), C.c_int(nthreads or default_threads())))
    return out


STE_OF, STE_DIFF = 1, 2


def gemm_ste_mask(A, B, prod_fmt, acc_fmt, order, chunk, kind, eps1=0.0, eps2=0.0, nthreads=0):
    """(mask1 uint32 [M][ceil(K/32)][N], mask2 uint32 [M][ceil(ceil(K/chunk)/32)][N] or None): STE bit of every
    FMAq step of the first hierarchy and, in chunked order, of every fold into the second (App. D)."""
    A, Ap = _u8(A)
    B, Bp = _u8(B)
    M, K = A.shape
    N, _ = B.shape
    pf, af = _fmt(prod_fmt), _fmt(acc_fmt)
    m1 = np.empty((M, (K + 31) // 32, N), dtype=np.uint32)
    m2 = None
    if order == 1:  # chunked
        m2 = np.empty((M, ((K + chunk - 1) // chunk + 31) // 32, N), dtype=np.uint32)
    u32 = C.POINTER(C.c_uint32)
    _check(lib().lbo_gemm_ste_mask(Ap, Bp, C.c_int64(M), C.c_int64(N), C.c_int64(K), C.byref(pf), C.byref(af),
                                   C.c_int(order), C.c_int64(chunk), C.c_int(kind), C.c_float(eps1), C.c_float(eps2),
                                   m1.ctypes.data_as(u32), m2.ctypes.data_as(u32) if m2 is not None else None,
                                   C.c_int(nthreads or default_threads())))
    return m1, m2


def conv_out_hw(H, W, KH, KW, stride, pad):
    sh, sw = stride
    ph, pw = pad
    return (H + 2 * ph - KH) // sh + 1, (W + 2 * pw - KW) // sw + 1


def conv2d(x, w, scale_x, scale_w, bias, stride, pad, prod_fmt, acc_fmt, order, chunk, nthreads=0):
    """x [B][H][W][Cin], w [Cout][KH][KW][Cin] (bytes) -> out [B][Hout][Wout][Cout]."""
    x, xp = _u8(x)
    w, wp = _u8(w)
    B, H, W, Cin = x.shape
    Cout, KH, KW, Cin2 = w.shape
    assert Cin == Cin2
    Hout, Wout = conv_out_hw(H, W, KH, KW, stride, pad)
    keep, sxp, sxl, swp, swl, bp = _scales(scale_x, scale_w, bias, B * Hout * Wout, Cout)
    pf, af = _fmt(prod_fmt), _fmt(acc_fmt)
    out = np.empty((B, max(Hout, 0), max(Wout, 0), Cout), dtype=np.float32)
    _check(lib().lbo_conv2d(xp, wp, sxp, C.c_int(sxl), swp, C.c_int(swl), bp, C.c_int64(B), C.c_int64(H),
                            C.c_int64(W), C.c_int64(Cin), C.c_int64(Cout), C.c_int64(KH), C.c_int64(KW),
                            C.c_int64(stride[0]), C.c_int64(stride[1]), C.c_int64(pad[0]), C.c_int64(pad[1]),
                            C.byref(pf), C.byref(af), C.c_int(order), C.c_int64(chunk),
                            out.ctypes.data_as(C.POINTER(C.c_float)), C.c_int(nthreads or default_threads())))
    return out


def conv2d_points(x, w, scale_x, scale_w, bias, stride, pad, prod_fmt, acc_fmt, order, chunk, ms, ns, nthreads=0):
    """Selected output scalars: ms[p] = (b*Hout + oh)*Wout + ow, ns[p] = output channel."""
    x, xp = _u8(x)
    w, wp = _u8(w)
    B, H, W, Cin = x.shape
    Cout, KH, KW, _ = w.shape
    Hout, Wout = conv_out_hw(H, W, KH, KW, stride, pad)
    keep, sxp, sxl, swp, swl, bp = _scales(scale_x, scale_w, bias, B * Hout * Wout, Cout)
    pf, af = _fmt(prod_fmt), _fmt(acc_fmt)
    ms, msp = _i64(ms)
    ns, nsp = _i64(ns)
    P = ms.size
    out = np.empty(P, dtype=np.float32)
    _check(lib().lbo_conv2d_points(xp, wp, sxp, C.c_int(sxl), swp, C.c_int(swl), bp, C.c_int64(B), C.c_int64(H),
                                   C.c_int64(W), C.c_int64(Cin), C.c_int64(Cout), C.c_int64(KH), C.c_int64(KW),
                                   C.c_int64(stride[0]), C.c_int64(stride[1]), C.c_int64(pad[0]),
                                   C.c_int64(pad[1]), C.byref(pf), C.byref(af), C.c_int(order), C.c_int64(chunk),
                                   msp, nsp, C.c_int64(P), out.ctypes.data_as(C.POINTER(C.c_float)),
                                   C.c_int(nthreads or default_threads())))
    return out
