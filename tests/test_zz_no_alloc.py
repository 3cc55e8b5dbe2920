"""lba_gemm_host_static: the host-buffer GEMM for callers that may not allocate device memory.

Some users of this library run where cudaMalloc is not an option: inside a server whose device memory was
carved up at start-up, in a plug-in that was handed buffers but no allocator, or in a loop where an allocation
would stall the whole device.  For them the library carries an 8 MiB workspace of its own.  This file checks,
through the C ABI, that the variant gives bit for bit what lba_gemm_host gives with a caller-supplied
workspace, and what the CPU oracle gives -- twice in a row, the second problem smaller and with other formats, so
that anything left in the shared workspace by the first call would show --, that no device memory is taken by the
first call or by a later one, that the accept/refuse boundary sits exactly at the 8 MiB, and that empty shapes are
accepted without any work.

It is collected last on purpose: a failure here cannot hide the result of any other test.  It needs nothing
from the tests before it and passes on its own in a fresh process.  Needs a B200.
"""
import numpy as np
import pytest
import torch

from oracle import lba_oracle as orc
from paper_2401_14110_b200 import binding as lba
from paper_2401_14110_b200 import synth, code_domain_formats, ORDER_SEQUENTIAL as SEQ, ORDER_CHUNKED as CHK

pytestmark = pytest.mark.gpu

DEV = "cuda:0"


def _bits(t):
    return t.numpy().view(np.uint32)


def _both_ways(M, N, K, config, fmts, order, with_bias):
    prod, acc = fmts
    A, sa, B, sb = synth.gemm_case(M, N, K, config=config)
    sb_cols = torch.linspace(0.5, 1.5, N) * sb
    bias = torch.linspace(-2, 2, N) if with_bias else None
    A, B = A.pin_memory(), B.pin_memory()
    # the existing entry point, workspace from the caller
    ws = torch.empty(lba.gemm_host_workspace_bytes(M, N, K, 1, N, with_bias), dtype=torch.uint8, device=DEV)
    want = torch.empty((M, N), dtype=torch.float32).pin_memory()
    lba.lba_gemm_host(A, B, sa, sb_cols, bias, prod, acc, order, 16, want, ws)
    torch.cuda.synchronize()
    # the variant under test: no workspace argument, nothing allocated on the device by the call
    got = torch.full((M, N), float("nan"), dtype=torch.float32).pin_memory()
    lba.lba_gemm_host_static(A, B, sa, sb_cols, bias, prod, acc, order, 16, got)
    torch.cuda.synchronize()
    assert np.array_equal(_bits(got), _bits(want)), f"{M}x{N}x{K}: built-in workspace result differs"
    ref = orc.gemm(A.numpy(), B.numpy(), sa.numpy(), sb_cols.numpy(), None if bias is None else bias.numpy(),
                   prod.as_tuple(), acc.as_tuple(), order, 16)
    assert np.array_equal(_bits(got), ref.view(np.uint32)), f"{M}x{N}x{K}: built-in workspace result differs from the oracle"


def _device_memory():
    free, _ = torch.cuda.mem_get_info()
    return free, torch.cuda.memory_allocated(), torch.cuda.memory_reserved()


def test_static_workspace_gemm_matches_caller_workspace_gemm_twice_in_a_row():
    _both_ways(300, 200, 160, config=71, fmts=code_domain_formats(7, 4), order=CHK, with_bias=True)
    _both_ways(130, 70, 48, config=72, fmts=code_domain_formats(4, 4, rounding=1), order=SEQ, with_bias=False)


def test_static_workspace_gemm_takes_no_device_memory():
    # the property the entry point exists for: no call of it allocates.  PyTorch's allocator must not see any of the
    # calls, the first included; the driver's free-memory figure must not move from the second call on (under lazy
    # module loading the driver may place the library's code and its built-in array only when they are first touched,
    # which is part of loading the library, not an allocation made by the call).
    prod, acc = code_domain_formats(7, 4)
    A, sa, B, sb = synth.gemm_case(96, 64, 64, config=73)
    A, B = A.pin_memory(), B.pin_memory()
    out = torch.empty((96, 64), dtype=torch.float32).pin_memory()
    torch.cuda.synchronize()
    torch_before = _device_memory()[1:]
    lba.lba_gemm_host_static(A, B, sa, sb, None, prod, acc, CHK, 16, out)
    torch.cuda.synchronize()
    assert _device_memory()[1:] == torch_before
    before = _device_memory()
    for _ in range(3):
        lba.lba_gemm_host_static(A, B, sa, sb, None, prod, acc, CHK, 16, out)
        torch.cuda.synchronize()
        assert _device_memory() == before


def test_static_workspace_boundary_and_empty_shapes():
    prod, acc = code_domain_formats(7, 4)
    one = torch.ones(1)
    # workspace need = up(M*K) + up(N*K) + 2 * 256 (scales) + up(4*M*N), each rounded up to 256 bytes
    K, N = 16, 1024
    M = 2029                            # 32512 + 16384 + 512 + 8310784 = 8360192 = 8 MiB - 28416: accepted
    assert lba.gemm_host_workspace_bytes(M, N, K, 1, 1, False) <= lba.STATIC_WORKSPACE_BYTES
    M_fit = max(m for m in range(2029, 2060) if lba.gemm_host_workspace_bytes(m, N, K, 1, 1, False) <= lba.STATIC_WORKSPACE_BYTES)
    assert lba.gemm_host_workspace_bytes(M_fit + 1, N, K, 1, 1, False) > lba.STATIC_WORKSPACE_BYTES
    for M_, ok in ((M_fit, True), (M_fit + 1, False)):
        A = torch.zeros((M_, K), dtype=torch.uint8)
        B = torch.zeros((N, K), dtype=torch.uint8)
        out = torch.full((M_, N), 7.0, dtype=torch.float32)
        if ok:
            lba.lba_gemm_host_static(A, B, one, one, None, prod, acc, CHK, 16, out)
            torch.cuda.synchronize()
            assert (out == 0).all()                      # all-zero operands: every output is +0
        else:
            with pytest.raises(lba.LbaError) as e:
                lba.lba_gemm_host_static(A, B, one, one, None, prod, acc, CHK, 16, out)
            assert e.value.status == -8
    # a need of exactly the limit is accepted, 256 bytes more is not: K = 0 leaves the two scales (512 bytes) and the
    # output, 4 * 32766 * 64 = 8 MiB - 512
    assert lba.gemm_host_workspace_bytes(32766, 64, 0, 1, 1, False) == lba.STATIC_WORKSPACE_BYTES
    assert lba.gemm_host_workspace_bytes(32767, 64, 0, 1, 1, False) == lba.STATIC_WORKSPACE_BYTES + 256
    out = torch.full((32766, 64), 7.0, dtype=torch.float32)
    lba.lba_gemm_host_static(torch.zeros((32766, 0), dtype=torch.uint8), torch.zeros((64, 0), dtype=torch.uint8), one, one,
                             None, prod, acc, CHK, 16, out)
    torch.cuda.synchronize()
    assert (out == 0).all()
    with pytest.raises(lba.LbaError) as e:
        lba.lba_gemm_host_static(torch.zeros((32767, 0), dtype=torch.uint8), torch.zeros((64, 0), dtype=torch.uint8), one,
                                 one, None, prod, acc, CHK, 16, torch.empty((32767, 64), dtype=torch.float32))
    assert e.value.status == -8
    # empty shapes: nothing to copy, nothing to launch, no error
    for (M_, N_, K_) in ((0, 8, 16), (8, 0, 16), (8, 8, 0)):
        A = torch.zeros((M_, K_), dtype=torch.uint8)
        B = torch.zeros((N_, K_), dtype=torch.uint8)
        out = torch.full((M_, N_), 7.0, dtype=torch.float32)
        lba.lba_gemm_host_static(A, B, one, one, None, prod, acc, CHK, 16, out)
        torch.cuda.synchronize()
        if K_ == 0:
            assert (out == 0).all()                      # an empty sum is +0


def test_static_workspace_gemm_refuses_what_does_not_fit():
    prod, acc = code_domain_formats(7, 4)
    M = N = 2048                    # the output alone is 16 MiB, the built-in workspace 8 MiB
    K = 16
    A = torch.zeros((M, K), dtype=torch.uint8)
    B = torch.zeros((N, K), dtype=torch.uint8)
    one = torch.ones(1)
    out = torch.empty((M, N), dtype=torch.float32)
    with pytest.raises(lba.LbaError) as e:
        lba.lba_gemm_host_static(A, B, one, one, None, prod, acc, CHK, 16, out)
    assert e.value.status == -8 and "built-in workspace" in str(e.value)
    assert lba.gemm_host_workspace_bytes(M, N, K, 1, 1, False) > lba.STATIC_WORKSPACE_BYTES
