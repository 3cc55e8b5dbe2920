"""The C ABI without a GPU: the library loads, exports every declared symbol, and rejects bad arguments
on the host before anything is enqueued."""
import ctypes as C
import os
import re

import pytest

from paper_2401_14110_b200 import binding as lba
from paper_2401_14110_b200 import LbaFormat, code_domain_formats, ORDER_CHUNKED as CHK, ORDER_SEQUENTIAL as SEQ

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared_functions():
    text = open(os.path.join(ROOT, "include", "lba.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(lba_[a-z0-9_]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    lib = lba.load_library()
    names = _declared_functions()
    assert "lba_gemm" in names and "lba_conv2d" in names and len(names) >= 10
    for name in names:
        assert getattr(lib, name) is not None
    assert sorted(lba.EXPORTS) == names
    assert lib.lba_version() == 1
    assert lib.lba_status_string(0) == b"ok"


def test_plan_selection_by_format_and_order():
    p, a = code_domain_formats(7, 4)
    assert "q=floor_fast" in lba.describe_plan(64, 64, 576, p, a, SEQ, 16)
    assert "order=seq" in lba.describe_plan(64, 64, 576, p, a, SEQ, 16)
    assert "order=chunk16" in lba.describe_plan(64, 64, 576, p, a, CHK, 16)
    assert "order=chunk_slab" in lba.describe_plan(64, 64, 576, p, a, CHK, 32)
    assert "order=chunk_any" in lba.describe_plan(64, 64, 576, p, a, CHK, 5)
    assert "order=seq" in lba.describe_plan(64, 64, 576, p, a, CHK, 576)       # one chunk == sequential
    assert "q=floor_full" in lba.describe_plan(64, 64, 576, LbaFormat(7, 4, 12), LbaFormat(7, 4, 10), CHK, 16)
    assert "q=floor_full" in lba.describe_plan(64, 64, 576, *code_domain_formats(4, 4), CHK, 16)
    assert "q=rne_full" in lba.describe_plan(64, 64, 576, *code_domain_formats(7, 4, rounding=1), CHK, 16)
    assert "q=rne_wide" in lba.describe_plan(64, 64, 576, LbaFormat(23, 8, 127, 1), LbaFormat(23, 8, 127, 1), SEQ, 16)
    assert "pq=none" in lba.describe_plan(64, 64, 576, p, a, CHK, 16)                # the product flush is reachable
    assert "pq=fused" in lba.describe_plan(64, 64, 576, *code_domain_formats(8, 6), CHK, 16)
    assert "pq=fused" in lba.describe_plan(64, 64, 576, *code_domain_formats(7, 4, flags=0), SEQ, 16)
    assert "pq=cut" in lba.describe_plan(64, 64, 576, *code_domain_formats(5, 6), CHK, 16)
    assert "load=conv_vec" in lba.describe_plan(64, 64, 576, p, a, CHK, 16, is_conv=True)
    assert "load=any" in lba.describe_plan(64, 64, 147, p, a, CHK, 16, is_conv=True, vec_ok=False)


@pytest.mark.parametrize("prod,acc,order,chunk,status", [
    (LbaFormat(0, 4, 8), LbaFormat(7, 4, 8), SEQ, 16, -3),
    (LbaFormat(7, 9, 8), LbaFormat(7, 4, 8), SEQ, 16, -3),
    (LbaFormat(7, 4, 500), LbaFormat(7, 4, 8), SEQ, 16, -3),
    (LbaFormat(7, 4, 8, 3), LbaFormat(7, 4, 8, 3), SEQ, 16, -3),
    (LbaFormat(7, 4, 8, 0), LbaFormat(7, 4, 8, 1), SEQ, 16, -3),          # mixed rounding rules
    (LbaFormat(22, 8, 127, 1), LbaFormat(22, 8, 127, 1), SEQ, 16, -3),    # nearest-even with M = 22
    (LbaFormat(7, 4, 8), LbaFormat(7, 4, 8), 2, 16, -4),
    (LbaFormat(7, 4, 8), LbaFormat(7, 4, 8), CHK, 0, -4),
])
def test_rejected_arguments(prod, acc, order, chunk, status):
    with pytest.raises(lba.LbaError) as e:
        lba.describe_plan(8, 8, 8, prod, acc, order, chunk)
    assert e.value.status == status


def test_host_side_checks_run_before_any_cuda_call():
    lib = lba.load_library()
    p, a = code_domain_formats(7, 4)
    pf, af = lba._fmt(p), lba._fmt(a)
    # null operands, negative sizes, bad scale lengths: all refused without touching a device
    assert lib.lba_gemm(None, None, None, 1, None, 1, None, 4, 4, 4, C.byref(pf), C.byref(af), 0, 16, None, None) == -1
    assert lib.lba_gemm(None, None, None, 1, None, 1, None, -1, 4, 4, C.byref(pf), C.byref(af), 0, 16, None, None) == -2
    fake = C.c_void_p(256)
    assert lib.lba_gemm(fake, fake, fake, 3, fake, 1, None, 4, 4, 4, C.byref(pf), C.byref(af), 0, 16, fake, None) == -5
    assert lib.lba_conv2d(fake, fake, fake, 1, fake, 1, None, 1, 2, 2, 3, 4, 5, 5, 1, 1, 0, 0, C.byref(pf),
                          C.byref(af), 0, 16, fake, None) == -2
    assert lib.lba_gemm_host_workspace_bytes(4, 4, 16, 1, 1, 0) == 256 * 5
    assert lib.lba_set_tile_override(9) == -2 and lib.lba_set_tile_override(-1) == 0


def test_host_variants_refuse_shapes_whose_byte_counts_would_wrap():
    # M*K, N*K and 4*M*N are formed in size_t inside the host-buffer variants: a shape for which one of them does
    # not fit must come back as an error code (and a workspace size of 0), never as a small wrapped size
    lib = lba.load_library()
    p, a = code_domain_formats(7, 4)
    pf, af = lba._fmt(p), lba._fmt(a)
    fake = C.c_void_p(256)
    huge = 1 << 62
    assert lib.lba_gemm_host_workspace_bytes(huge, 1, 4, 1, 1, 0) == 0          # M*K = 2^64
    assert lib.lba_gemm_host_workspace_bytes(1 << 31, 1 << 31, 16, 1, 1, 0) == 0  # 4*M*N = 2^64
    assert lib.lba_gemm_host_workspace_bytes(1 << 20, 1 << 20, 16, 1, 1, 0) > 0   # 4 TiB: large, but it fits
    for (M, N, K) in ((huge, 1, 4), (1 << 31, 1 << 31, 16), (4, 4, 1 << 31)):
        assert lib.lba_gemm_host(fake, fake, fake, 1, fake, 1, None, M, N, K, C.byref(pf), C.byref(af), 1, 16, fake, fake,
                                 C.c_size_t(1 << 40), None) == -2
        assert lib.lba_gemm_host_static(fake, fake, fake, 1, fake, 1, None, M, N, K, C.byref(pf), C.byref(af), 1, 16, fake,
                                        None) in (-2, -8)
    # convolution: the output byte count is guarded the same way
    assert lib.lba_conv2d_host_workspace_bytes(1 << 20, 1, 1, 1, 1 << 20, 1, 1, 1, 1, 0, 0, 1, 1, 0) > 0
    assert lib.lba_conv2d_host_workspace_bytes(1 << 30, 1, 1, 1, 1 << 30, 1, 1, 1, 1, 0, 0, 1, 1, 0) == 0     # 4*M*C_out = 2^62


def test_tile_choice_follows_the_measured_order():
    # the host's tile model is fitted to measurements on B200 (148 SMs is also what the model assumes without a device):
    # these are the shapes it was fitted and checked on, with the tile that measured fastest
    f, r = code_domain_formats(7, 4), code_domain_formats(7, 4, rounding=1)
    tile = lambda shape, fm, order: lba.describe_plan(*shape, *fm, order, 16).split(" q=")[0]
    assert tile((8192, 8192, 8192), f, CHK) == "tile=128x128x16 micro=8x8"       # full SMs, floor: the 8x8 micro-tile
    assert tile((8192, 8192, 8192), f, SEQ) == "tile=128x128x16 micro=8x8"
    assert tile((8192, 8192, 8192), r, CHK) == "tile=64x64x16 micro=4x8"         # nearest-even, chunk 16: 64x64 is 12 % faster
    assert tile((4096, 768, 768), f, CHK) == "tile=64x64x16 micro=4x8"           # BERT linears: not the 32x32 tile
    assert tile((25088, 128, 1152), f, CHK) == "tile=64x64x16 micro=4x8"         # ResNet-18 layer2
    assert tile((1568, 512, 4608), f, CHK) == "tile=64x64x16 pair micro=4x8"     # layer4: two CTAs per tile
    assert tile((1568, 512, 4608), f, SEQ) == "tile=32x32x16 micro=4x4"          # no chunks to share in sequential order
    assert tile((32, 1000, 512), f, CHK) == "tile=32x32x16 micro=4x4"            # the classifier


def test_describe_plan_for_batched_calls():
    # 384 problems of 128x128 fill the SMs with 64x64 tiles; one such problem alone would get the 32x32 tile
    f = code_domain_formats(7, 4)
    assert lba.describe_plan(128, 128, 64, *f, CHK, 16).startswith("tile=32x32x16")
    assert lba.describe_plan(128, 128, 64, *f, CHK, 16, batch=384).startswith("tile=64x64x16 micro=4x8")
    with pytest.raises(lba.LbaError):
        lba.describe_plan(128, 128, 64, *f, CHK, 16, batch=0)
