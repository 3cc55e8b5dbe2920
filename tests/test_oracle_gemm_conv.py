"""Pins for the oracle's GEMM and convolution indexing and the scaling epilogue.  CPU only."""
import numpy as np
import pytest
import torch
import torch.nn.functional as F

from oracle import lba_oracle as orc
from paper_2401_14110_b200 import synth

SEQ, CHK = orc.SEQUENTIAL, orc.CHUNKED
PROD, ACC = (7, 4, -2, 0, 1), (7, 4, -4, 0, 1)
EXACT = (12, 6, 20, 0, 1)     # with small-integer inputs nothing is ever rounded in this format


def _dec(codes):
    return synth.e4m3_decode(torch.from_numpy(np.ascontiguousarray(codes)))


def test_gemm_is_the_dot_product_of_row_pairs():
    # App. A: Y = X W^T, y = Y_kl uses x_i = X_ki, w_i = W_li
    A = synth.random_codes((5, 37), 1).numpy()
    B = synth.random_codes((7, 37), 2).numpy()
    for order, chunk in ((SEQ, 16), (CHK, 16)):
        out = orc.gemm(A, B, 1.0, 1.0, None, PROD, ACC, order, chunk)
        assert out.shape == (5, 7)
        for m in range(5):
            for n in range(7):
                assert float(out[m, n]) == orc.dot(PROD, ACC, order, chunk, A[m], B[n])


def test_gemm_exact_case_matches_integer_matmul():
    A = synth.small_integer_codes((9, 50), 3, max_abs=4).numpy()
    B = synth.small_integer_codes((6, 50), 4, max_abs=4).numpy()
    want = _dec(A).to(torch.int64) @ _dec(B).to(torch.int64).T
    out = orc.gemm(A, B, 1.0, 1.0, None, EXACT, EXACT, CHK, 16)
    assert np.array_equal(out.astype(np.int64), want.numpy())


def test_points_match_full_gemm():
    A = synth.random_codes((20, 64), 5).numpy()
    B = synth.random_codes((30, 64), 6).numpy()
    sa = np.linspace(0.5, 1.5, 20).astype(np.float32)
    sb = np.linspace(0.01, 0.02, 30).astype(np.float32)
    bias = np.linspace(-1, 1, 30).astype(np.float32)
    full = orc.gemm(A, B, sa, sb, bias, PROD, ACC, CHK, 16)
    ms, ns = synth.sample_tiles(20, 30, 3, 4, 7)
    pts = orc.gemm_points(A, B, sa, sb, bias, PROD, ACC, CHK, 16, ms, ns)
    assert np.array_equal(pts, full[ms, ns])
    # thread count does not change anything
    assert np.array_equal(full, orc.gemm(A, B, sa, sb, bias, PROD, ACC, CHK, 16, nthreads=1))


def test_epilogue_is_three_binary32_operations():
    A = synth.random_codes((6, 48), 8).numpy()
    B = synth.random_codes((5, 48), 9).numpy()
    y = orc.gemm(A, B, 1.0, 1.0, None, PROD, ACC, SEQ, 16)
    sa = np.array([0.1, 0.3, 0.7, 1.1, 1.3, 1.7], np.float32)
    sb = np.array([0.013, 0.017, 0.019, 0.023, 0.029], np.float32)
    bias = np.array([0.5, -0.25, 3.0, 1e-3, -7.0], np.float32)
    want = (y * sa[:, None]).astype(np.float32)
    want = (want * sb[None, :]).astype(np.float32)
    assert np.array_equal(orc.gemm(A, B, sa, sb, None, PROD, ACC, SEQ, 16), want)
    assert np.array_equal(orc.gemm(A, B, sa, sb, bias, PROD, ACC, SEQ, 16), (want + bias[None, :]).astype(np.float32))
    one = orc.gemm(A, B, np.float32(0.37), np.float32(0.011), None, PROD, ACC, SEQ, 16)
    assert np.array_equal(one, ((y * np.float32(0.37)).astype(np.float32) * np.float32(0.011)).astype(np.float32))


def _patches(x_codes, KH, KW, stride, pad):
    """im2col by torch.nn.functional.unfold, reordered to k = (kh, kw, c_in); padded taps become code 0."""
    B, H, W, C = x_codes.shape
    xf = torch.from_numpy(x_codes).permute(0, 3, 1, 2).to(torch.float32)        # codes as numbers, NCHW
    cols = F.unfold(xf, (KH, KW), padding=pad, stride=stride)                    # [B][C*KH*KW][L], c slowest
    L = cols.shape[-1]
    cols = cols.reshape(B, C, KH, KW, L).permute(0, 4, 2, 3, 1).reshape(B * L, KH * KW * C)
    return cols.to(torch.uint8).numpy()


CONV_CASES = [
    # B, H, W, Cin, Cout, KH, KW, stride, pad
    (2, 9, 8, 3, 5, 3, 3, (1, 1), (1, 1)),
    (1, 11, 11, 3, 4, 7, 7, (2, 2), (3, 3)),
    (2, 8, 8, 16, 6, 1, 1, (2, 2), (0, 0)),
    (1, 7, 9, 5, 3, 3, 2, (2, 1), (0, 2)),
    (1, 6, 6, 32, 8, 3, 3, (2, 2), (1, 1)),
]


@pytest.mark.parametrize("case", CONV_CASES)
def test_conv_equals_gemm_on_gathered_patches(case):
    B, H, W, Cin, Cout, KH, KW, stride, pad = case
    x = synth.random_codes((B, H, W, Cin), 11).numpy()
    w = synth.random_codes((Cout, KH, KW, Cin), 12).numpy()
    sw = np.linspace(0.5, 2.0, Cout).astype(np.float32)
    bias = np.linspace(-3, 3, Cout).astype(np.float32)
    Hout, Wout = orc.conv_out_hw(H, W, KH, KW, stride, pad)
    for order, chunk in ((SEQ, 16), (CHK, 16)):
        out = orc.conv2d(x, w, 0.25, sw, bias, stride, pad, PROD, ACC, order, chunk)
        assert out.shape == (B, Hout, Wout, Cout)
        A = _patches(x, KH, KW, stride, pad)
        ref = orc.gemm(A, w.reshape(Cout, -1), 0.25, sw, bias, PROD, ACC, order, chunk)
        assert np.array_equal(out.reshape(-1, Cout), ref)
    ms = np.array([0, B * Hout * Wout - 1, (B * Hout * Wout) // 2], np.int64)
    ns = np.array([Cout - 1, 0, Cout // 2], np.int64)
    pts = orc.conv2d_points(x, w, 0.25, sw, bias, stride, pad, PROD, ACC, CHK, 16, ms, ns)
    assert np.array_equal(pts, out.reshape(-1, Cout)[ms, ns])


@pytest.mark.parametrize("case", CONV_CASES)
def test_conv_exact_case_matches_torch_conv2d(case):
    B, H, W, Cin, Cout, KH, KW, stride, pad = case
    x = synth.small_integer_codes((B, H, W, Cin), 13, max_abs=3).numpy()
    w = synth.small_integer_codes((Cout, KH, KW, Cin), 14, max_abs=3).numpy()
    want = F.conv2d(_dec(x).permute(0, 3, 1, 2).double(), _dec(w).permute(0, 3, 1, 2).double(), stride=stride,
                    padding=pad).permute(0, 2, 3, 1)
    out = orc.conv2d(x, w, 1.0, 1.0, None, stride, pad, EXACT, EXACT, CHK, 16)
    assert np.array_equal(out.astype(np.float64), want.numpy())


def test_pointwise_conv_is_a_gemm():
    x = synth.random_codes((2, 5, 5, 24), 15).numpy()
    w = synth.random_codes((7, 1, 1, 24), 16).numpy()
    out = orc.conv2d(x, w, 1.0, 1.0, None, (1, 1), (0, 0), PROD, ACC, CHK, 16)
    ref = orc.gemm(x.reshape(-1, 24), w.reshape(7, 24), 1.0, 1.0, None, PROD, ACC, CHK, 16)
    assert np.array_equal(out.reshape(-1, 7), ref)


def test_error_statuses():
    A = synth.random_codes((2, 8), 17).numpy()
    bad = A.copy()
    bad[1, 3] = 0x7F
    with pytest.raises(orc.OracleError) as e:
        orc.gemm(bad, A, 1.0, 1.0, None, PROD, ACC, SEQ, 16)
    assert e.value.status == -3
    with pytest.raises(orc.OracleError):
        orc.gemm(A, A, 1.0, 1.0, None, PROD, ACC, 2, 16)
    with pytest.raises(orc.OracleError):
        orc.gemm(A, A, 1.0, 1.0, None, PROD, ACC, CHK, 0)
    x = synth.random_codes((1, 2, 2, 3), 18).numpy()
    w = synth.random_codes((1, 5, 5, 3), 19).numpy()
    with pytest.raises(orc.OracleError):
        orc.conv2d(x, w, 1.0, 1.0, None, (1, 1), (0, 0), PROD, ACC, SEQ, 16)
    # empty problems are legal and return empty outputs
    assert orc.gemm(A[:0], A, 1.0, 1.0, None, PROD, ACC, SEQ, 16).shape == (0, 2)
    z = orc.gemm(A[:, :0], A[:, :0], 1.0, 1.0, None, PROD, ACC, SEQ, 16)
    assert z.shape == (2, 2) and np.all(z == 0) and not np.any(np.signbit(z))
