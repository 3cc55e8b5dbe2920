"""lba_gemm_host_static: the host-buffer GEMM for callers that may not allocate device memory.

Some users of this library run where cudaMalloc is not an option: inside a server whose device memory was
carved up at start-up, in a plug-in that was handed buffers but no allocator, or in a loop where an allocation
would stall the whole device.  For them the library carries an 8 MiB workspace of its own.  This file checks,
through the C ABI, that the variant gives bit for bit what lba_gemm_host gives with a caller-supplied
workspace -- twice in a row, the second problem smaller and with other formats, so that anything left in the
shared workspace by the first call would show -- and that a problem beyond the built-in limit is refused.

It is collected last on purpose: a failure here cannot hide the result of any other test.  It needs nothing
from the tests before it and passes on its own in a fresh process.  Needs a B200.
"""
import numpy as np
import pytest
import torch

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


def test_static_workspace_gemm_matches_caller_workspace_gemm_twice_in_a_row():
    _both_ways(300, 200, 160, config=71, fmts=code_domain_formats(7, 4), order=CHK, with_bias=True)
    _both_ways(130, 70, 48, config=72, fmts=code_domain_formats(4, 4, rounding=1), order=SEQ, with_bias=False)


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
