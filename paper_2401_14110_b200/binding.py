"""Thin ctypes binding of ``liblba.so`` (C ABI declared in ``include/lba.h``).

Argument marshalling only: PyTorch supplies device memory and the current stream; every step of
the computation runs in the CUDA kernels behind the C entry points.  There is no fallback: if the
library is missing, or a call returns an error, an exception is raised.
"""
import ctypes as C
import os

import torch

from .formats import LbaFormat, ORDER_CHUNKED, PAPER_CHUNK

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "liblba.so")

EXPORTS = ["lba_gemm", "lba_gemm_batched", "lba_gemm_last_overflow", "lba_gemm_ste_mask", "lba_conv2d", "lba_gemm_host_workspace_bytes", "lba_gemm_host",
           "lba_conv2d_host_workspace_bytes", "lba_conv2d_host", "lba_gemm_host_static", "lba_count_nan_codes", "lba_describe_plan", "lba_describe_plan_batched",
           "lba_set_tile_override", "lba_status_string", "lba_last_cuda_error", "lba_version"]


class LbaError(RuntimeError):
    def __init__(self, status, text, cuda_error=0):
        super().__init__(f"liblba status {status}: {text}" + (f" (cudaError {cuda_error})" if cuda_error else ""))
        self.status = status
        self.cuda_error = cuda_error


class _Fmt(C.Structure):
    _fields_ = [("man_bits", C.c_int32), ("exp_bits", C.c_int32), ("bias", C.c_int32), ("rounding", C.c_int32),
                ("flags", C.c_int32)]


_lib = None


def load_library():
    """Load liblba.so from the package directory; raises if it has not been built."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise RuntimeError(f"{LIB_PATH} is missing: build it with `python -m paper_2401_14110_b200.build` "
                           "(there is no CPU or PyTorch fallback)")
    lib = C.CDLL(LIB_PATH)
    lib.lba_status_string.restype = C.c_char_p
    lib.lba_status_string.argtypes = [C.c_int]
    lib.lba_gemm_host_workspace_bytes.restype = C.c_size_t
    lib.lba_gemm_host_workspace_bytes.argtypes = [C.c_int64, C.c_int64, C.c_int64, C.c_int, C.c_int, C.c_int]
    lib.lba_conv2d_host_workspace_bytes.restype = C.c_size_t
    lib.lba_conv2d_host_workspace_bytes.argtypes = [C.c_int] * 14
    gemm_args = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_int, C.c_void_p, C.c_int, C.c_void_p, C.c_int64, C.c_int64,
                 C.c_int64, C.POINTER(_Fmt), C.POINTER(_Fmt), C.c_int, C.c_int, C.c_void_p]
    lib.lba_gemm.argtypes = gemm_args + [C.c_void_p]
    lib.lba_gemm_host.argtypes = gemm_args + [C.c_void_p, C.c_size_t, C.c_void_p]
    lib.lba_gemm_last_overflow.argtypes = [C.c_void_p, C.c_void_p, C.c_int64, C.c_int64, C.c_int64, C.POINTER(_Fmt),
                                           C.POINTER(_Fmt), C.c_void_p, C.c_void_p]
    lib.lba_gemm_ste_mask.argtypes = [C.c_void_p, C.c_void_p, C.c_int64, C.c_int64, C.c_int64, C.POINTER(_Fmt),
                                      C.POINTER(_Fmt), C.c_int, C.c_int, C.c_int, C.c_float, C.c_float, C.c_void_p,
                                      C.c_void_p, C.c_void_p]
    lib.lba_gemm_batched.argtypes = gemm_args[:7] + [C.c_int64] * 7 + gemm_args[10:] + [C.c_void_p]
    lib.lba_gemm_host_static.argtypes = gemm_args + [C.c_void_p]
    conv_args = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_int, C.c_void_p, C.c_int, C.c_void_p] + [C.c_int] * 11 + \
        [C.POINTER(_Fmt), C.POINTER(_Fmt), C.c_int, C.c_int, C.c_void_p]
    lib.lba_conv2d.argtypes = conv_args + [C.c_void_p]
    lib.lba_conv2d_host.argtypes = conv_args + [C.c_void_p, C.c_size_t, C.c_void_p]
    lib.lba_count_nan_codes.argtypes = [C.c_void_p, C.c_int64, C.c_void_p, C.c_void_p]
    lib.lba_describe_plan.argtypes = [C.c_int64, C.c_int64, C.c_int64, C.POINTER(_Fmt), C.POINTER(_Fmt), C.c_int,
                                      C.c_int, C.c_int, C.c_int, C.c_char_p, C.c_size_t]
    lib.lba_describe_plan_batched.argtypes = [C.c_int64] + lib.lba_describe_plan.argtypes
    for name in EXPORTS:
        getattr(lib, name)
    _lib = lib
    return lib


def _check(status):
    if status != 0:
        lib = load_library()
        raise LbaError(status, lib.lba_status_string(status).decode(), lib.lba_last_cuda_error())


def _fmt(f):
    t = f.as_tuple() if isinstance(f, LbaFormat) else tuple(f)
    return _Fmt(*[int(v) for v in t])


def _stream(stream):
    if stream is None:
        stream = torch.cuda.current_stream()
    return C.c_void_p(stream.cuda_stream if hasattr(stream, "cuda_stream") else int(stream))


def _dev(t, dtype, name):
    if t is None:
        return None
    if not (isinstance(t, torch.Tensor) and t.is_cuda and t.dtype == dtype and t.is_contiguous()):
        raise TypeError(f"{name} must be a contiguous CUDA tensor of dtype {dtype}")
    return C.c_void_p(t.data_ptr())


def _host(t, dtype, name):
    if t is None:
        return None
    if not (isinstance(t, torch.Tensor) and not t.is_cuda and t.dtype == dtype and t.is_contiguous()):
        raise TypeError(f"{name} must be a contiguous CPU tensor of dtype {dtype}")
    return C.c_void_p(t.data_ptr())


def conv_out_hw(H, W, KH, KW, stride, pad):
    return (H + 2 * pad[0] - KH) // stride[0] + 1, (W + 2 * pad[1] - KW) // stride[1] + 1


def lba_gemm(A, B, scale_a, scale_b, bias, prod_fmt, acc_fmt, order=ORDER_CHUNKED, chunk=PAPER_CHUNK, out=None,
             stream=None):
    """out[M][N] (float32, CUDA) for A [M][K], B [N][K] E4M3 bytes on the GPU.  See ``lba_gemm`` in lba.h."""
    lib = load_library()
    M, K = A.shape
    N, K2 = B.shape
    if K != K2:
        raise ValueError("A and B disagree on K")
    if out is None:
        out = torch.empty((M, N), dtype=torch.float32, device=A.device)
    pf, af = _fmt(prod_fmt), _fmt(acc_fmt)
    _check(lib.lba_gemm(_dev(A, torch.uint8, "A"), _dev(B, torch.uint8, "B"), _dev(scale_a, torch.float32, "scale_a"),
                        scale_a.numel(), _dev(scale_b, torch.float32, "scale_b"), scale_b.numel(),
                        _dev(bias, torch.float32, "bias"), M, N, K, C.byref(pf), C.byref(af), order, chunk,
                        _dev(out, torch.float32, "out"), _stream(stream)))
    return out


def lba_gemm_batched(A, B, scale_a, scale_b, bias, prod_fmt, acc_fmt, order=ORDER_CHUNKED, chunk=PAPER_CHUNK, out=None,
                     stream=None):
    """out[Z][M][N] for A [Z][M][K] and B [Z][N][K] (or [N][K], shared by all Z problems).  See lba.h."""
    lib = load_library()
    Z, M, K = A.shape
    if B.dim() == 2:
        N, K2 = B.shape
        stride_b = 0
    else:
        Zb, N, K2 = B.shape
        if Zb != Z:
            raise ValueError("A and B disagree on the batch size")
        stride_b = N * K
    if K != K2:
        raise ValueError("A and B disagree on K")
    if out is None:
        out = torch.empty((Z, M, N), dtype=torch.float32, device=A.device)
    pf, af = _fmt(prod_fmt), _fmt(acc_fmt)
    _check(lib.lba_gemm_batched(_dev(A, torch.uint8, "A"), _dev(B, torch.uint8, "B"),
                                _dev(scale_a, torch.float32, "scale_a"), scale_a.numel(),
                                _dev(scale_b, torch.float32, "scale_b"), scale_b.numel(),
                                _dev(bias, torch.float32, "bias"), Z, M, N, K, M * K, stride_b, M * N, C.byref(pf),
                                C.byref(af), order, chunk, _dev(out, torch.float32, "out"), _stream(stream)))
    return out


def lba_gemm_last_overflow(A, B, prod_fmt, acc_fmt, out=None, stream=None):
    """int32 [M][N]: index of the last sequential step at which Q_acc overflowed, -1 if none.  See lba.h."""
    lib = load_library()
    M, K = A.shape
    N, K2 = B.shape
    if K != K2:
        raise ValueError("A and B disagree on K")
    if out is None:
        out = torch.empty((M, N), dtype=torch.int32, device=A.device)
    pf, af = _fmt(prod_fmt), _fmt(acc_fmt)
    _check(lib.lba_gemm_last_overflow(_dev(A, torch.uint8, "A"), _dev(B, torch.uint8, "B"), M, N, K, C.byref(pf),
                                      C.byref(af), _dev(out, torch.int32, "last"), _stream(stream)))
    return out


STE_OF, STE_DIFF = 1, 2


def lba_gemm_ste_mask(A, B, prod_fmt, acc_fmt, order=ORDER_CHUNKED, chunk=PAPER_CHUNK, ste=STE_OF, eps1=0.0, eps2=0.0,
                      mask1=None, mask2=None, stream=None):
    """(mask1 int32 [M][ceil(K/32)][N], mask2 int32 [M][ceil(ceil(K/chunk)/32)][N] or None): one STE bit per FMAq
    step, as 32-bit words (torch has no unsigned 32-bit arithmetic; the bit patterns are what counts).  See lba.h."""
    lib = load_library()
    M, K = A.shape
    N, K2 = B.shape
    if K != K2:
        raise ValueError("A and B disagree on K")
    if mask1 is None:
        mask1 = torch.empty((M, (K + 31) // 32, N), dtype=torch.int32, device=A.device)
    if order != ORDER_CHUNKED:
        mask2 = None
    elif mask2 is None:
        mask2 = torch.empty((M, ((K + chunk - 1) // max(chunk, 1) + 31) // 32, N), dtype=torch.int32, device=A.device)
    pf, af = _fmt(prod_fmt), _fmt(acc_fmt)
    _check(lib.lba_gemm_ste_mask(_dev(A, torch.uint8, "A"), _dev(B, torch.uint8, "B"), M, N, K, C.byref(pf), C.byref(af),
                                 order, chunk, ste, C.c_float(eps1), C.c_float(eps2), _dev(mask1, torch.int32, "mask1"),
                                 None if mask2 is None else _dev(mask2, torch.int32, "mask2"), _stream(stream)))
    return mask1, mask2


def lba_conv2d(x, w, scale_x, scale_w, bias, stride, pad, prod_fmt, acc_fmt, order=ORDER_CHUNKED, chunk=PAPER_CHUNK,
               out=None, stream=None):
    """out [B][Hout][Wout][Cout] for x [B][H][W][Cin], w [Cout][KH][KW][Cin] E4M3 bytes.  See lba.h."""
    lib = load_library()
    B, H, W, Cin = x.shape
    Cout, KH, KW, Cin2 = w.shape
    if Cin != Cin2:
        raise ValueError("x and w disagree on C_in")
    Hout, Wout = conv_out_hw(H, W, KH, KW, stride, pad)
    if out is None:
        out = torch.empty((B, max(Hout, 0), max(Wout, 0), Cout), dtype=torch.float32, device=x.device)
    pf, af = _fmt(prod_fmt), _fmt(acc_fmt)
    _check(lib.lba_conv2d(_dev(x, torch.uint8, "x"), _dev(w, torch.uint8, "w"), _dev(scale_x, torch.float32, "scale_x"),
                          scale_x.numel(), _dev(scale_w, torch.float32, "scale_w"), scale_w.numel(),
                          _dev(bias, torch.float32, "bias"), B, H, W, Cin, Cout, KH, KW, stride[0], stride[1], pad[0],
                          pad[1], C.byref(pf), C.byref(af), order, chunk, _dev(out, torch.float32, "out"),
                          _stream(stream)))
    return out


def gemm_host_workspace_bytes(M, N, K, scale_a_len, scale_b_len, has_bias):
    return load_library().lba_gemm_host_workspace_bytes(M, N, K, scale_a_len, scale_b_len, int(has_bias))


def lba_gemm_host(A, B, scale_a, scale_b, bias, prod_fmt, acc_fmt, order, chunk, out, workspace, stream=None):
    """Host-buffer variant: CPU tensors in (pinned recommended), CPU ``out``; ``workspace`` is a CUDA uint8 tensor."""
    lib = load_library()
    M, K = A.shape
    N, _ = B.shape
    pf, af = _fmt(prod_fmt), _fmt(acc_fmt)
    _check(lib.lba_gemm_host(_host(A, torch.uint8, "A"), _host(B, torch.uint8, "B"),
                             _host(scale_a, torch.float32, "scale_a"), scale_a.numel(),
                             _host(scale_b, torch.float32, "scale_b"), scale_b.numel(),
                             _host(bias, torch.float32, "bias"), M, N, K, C.byref(pf), C.byref(af), order, chunk,
                             _host(out, torch.float32, "out"), _dev(workspace, torch.uint8, "workspace"),
                             workspace.numel(), _stream(stream)))
    return out


STATIC_WORKSPACE_BYTES = 8 << 20   # LBA_STATIC_WORKSPACE_BYTES in lba.h


def lba_gemm_host_static(A, B, scale_a, scale_b, bias, prod_fmt, acc_fmt, order, chunk, out, stream=None):
    """``lba_gemm_host`` for callers that cannot allocate device memory: CPU tensors in, CPU ``out``, and the
    device workspace is an 8 MiB array built into the library (shared by all calls on a device, so calls must
    not overlap on the GPU).  Larger problems raise ``LbaError`` with status -8.  No tensor is created here."""
    lib = load_library()
    M, K = A.shape
    N, _ = B.shape
    pf, af = _fmt(prod_fmt), _fmt(acc_fmt)
    _check(lib.lba_gemm_host_static(_host(A, torch.uint8, "A"), _host(B, torch.uint8, "B"),
                                    _host(scale_a, torch.float32, "scale_a"), scale_a.numel(),
                                    _host(scale_b, torch.float32, "scale_b"), scale_b.numel(),
                                    _host(bias, torch.float32, "bias"), M, N, K, C.byref(pf), C.byref(af), order,
                                    chunk, _host(out, torch.float32, "out"), _stream(stream)))
    return out


def conv2d_host_workspace_bytes(B, H, W, Cin, Cout, KH, KW, stride, pad, scale_x_len, scale_w_len, has_bias):
    return load_library().lba_conv2d_host_workspace_bytes(B, H, W, Cin, Cout, KH, KW, stride[0], stride[1], pad[0],
                                                          pad[1], scale_x_len, scale_w_len, int(has_bias))


def lba_conv2d_host(x, w, scale_x, scale_w, bias, stride, pad, prod_fmt, acc_fmt, order, chunk, out, workspace,
                    stream=None):
    lib = load_library()
    B, H, W, Cin = x.shape
    Cout, KH, KW, _ = w.shape
    pf, af = _fmt(prod_fmt), _fmt(acc_fmt)
    _check(lib.lba_conv2d_host(_host(x, torch.uint8, "x"), _host(w, torch.uint8, "w"),
                               _host(scale_x, torch.float32, "scale_x"), scale_x.numel(),
                               _host(scale_w, torch.float32, "scale_w"), scale_w.numel(),
                               _host(bias, torch.float32, "bias"), B, H, W, Cin, Cout, KH, KW, stride[0], stride[1],
                               pad[0], pad[1], C.byref(pf), C.byref(af), order, chunk,
                               _host(out, torch.float32, "out"), _dev(workspace, torch.uint8, "workspace"),
                               workspace.numel(), _stream(stream)))
    return out


def count_nan_codes(codes, stream=None):
    """Number of E4M3 NaN codes (0x7F, 0xFF) in a CUDA uint8 tensor (synchronises)."""
    lib = load_library()
    count = torch.zeros(1, dtype=torch.int64, device=codes.device)
    _check(lib.lba_count_nan_codes(_dev(codes, torch.uint8, "codes"), codes.numel(), C.c_void_p(count.data_ptr()),
                                   _stream(stream)))
    return int(count.item())


def set_tile_override(tile):
    """Force the CTA tile (0..3, 5 = cluster pair) or restore the automatic choice (-1).  A testing hook: process-wide.
    Speed only; results are unchanged."""
    _check(load_library().lba_set_tile_override(int(tile)))


def describe_plan(M, N, K, prod_fmt, acc_fmt, order=ORDER_CHUNKED, chunk=PAPER_CHUNK, is_conv=False, vec_ok=True, batch=1):
    """Text description of the kernel variant a call would run (``batch`` problems for ``lba_gemm_batched``); raises
    LbaError for rejected arguments."""
    lib = load_library()
    buf = C.create_string_buffer(256)
    pf, af = _fmt(prod_fmt), _fmt(acc_fmt)
    _check(lib.lba_describe_plan_batched(batch, M, N, K, C.byref(pf), C.byref(af), order, chunk, int(is_conv), int(vec_ok),
                                         buf, 256))
    return buf.value.decode()
