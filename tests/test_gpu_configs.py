"""The five benchmark configurations at full size: CUDA path versus the CPU oracle, bit for bit, on sampled outputs.

Every contraction runs at its full shape in the launch configuration the benchmark times (automatic tile
choice); the oracle then recomputes seeded 16x16 output tiles, plus, for convolutions, output positions whose
receptive field touches the padded border, from the very bytes the GPU call read.  Needs a B200.
"""
import numpy as np
import pytest
import torch

from oracle import lba_oracle as orc
from paper_2401_14110_b200 import binding as lba
from helpers.fmt_range import r_of, r_uf
from paper_2401_14110_b200 import synth, workloads
from paper_2401_14110_b200 import code_domain_formats, m4e3_input_formats, fixed_point_format, ORDER_SEQUENTIAL as SEQ, ORDER_CHUNKED as CHK

pytestmark = pytest.mark.gpu

DEV = "cuda:0"


def _bits(a):
    return np.ascontiguousarray(a, dtype=np.float32).view(np.uint32).reshape(-1)


def _assert_points_equal(out_2d, ms, ns, want, what):
    got = out_2d[torch.from_numpy(ms).to(out_2d.device), torch.from_numpy(ns).to(out_2d.device)].cpu().numpy()
    bad = np.nonzero(_bits(got) != _bits(want))[0]
    assert bad.size == 0, (f"{what}: {bad.size} of {got.size} sampled outputs differ; first at (m={ms[bad[0]]}, "
                           f"n={ns[bad[0]]}): gpu={got[bad[0]]!r} oracle={want[bad[0]]!r}")


def _border_points(call, n_points, seed):
    """Output positions (b, 0 or last, *) and (b, *, 0 or last): their windows overlap the zero padding."""
    b, h, w, _ = call.x.shape
    cout, kh, kw, _ = call.w.shape
    ho, wo = lba.conv_out_hw(h, w, kh, kw, call.stride, call.pad)
    g = torch.Generator().manual_seed(seed)
    bb = torch.randint(0, b, (n_points,), generator=g)
    edge = torch.randint(0, 4, (n_points,), generator=g)
    along_h = torch.randint(0, ho, (n_points,), generator=g)
    along_w = torch.randint(0, wo, (n_points,), generator=g)
    oh = torch.where(edge == 0, torch.zeros_like(along_h), torch.where(edge == 1, torch.full_like(along_h, ho - 1), along_h))
    ow = torch.where(edge == 2, torch.zeros_like(along_w), torch.where(edge == 3, torch.full_like(along_w, wo - 1), along_w))
    ms = ((bb * ho + oh) * wo + ow).numpy().astype(np.int64)
    ns = torch.randint(0, cout, (n_points,), generator=g).numpy().astype(np.int64)
    return ms, ns


def _check_call(call, prod, acc, order, tiles, seed):
    m, n, k = call.gemm_shape
    out = torch.empty((m, n), dtype=torch.float32, device=DEV)
    ms, ns = synth.sample_tiles(m, n, tiles, 16, seed)
    if call.kind == "conv":
        b, h, w, _ = call.x.shape
        cout, kh, kw, _ = call.w.shape
        ho, wo = lba.conv_out_hw(h, w, kh, kw, call.stride, call.pad)
        lba.lba_conv2d(call.x, call.w, call.sx, call.sw, None, call.stride, call.pad, prod, acc, order, 16,
                       out=out.view(b, ho, wo, cout))
        if call.pad != (0, 0):
            bm, bn = _border_points(call, 2048, seed + 1)
            ms, ns = np.concatenate([ms, bm]), np.concatenate([ns, bn])
        want = orc.conv2d_points(call.x.cpu().numpy(), call.w.cpu().numpy(), call.sx.cpu().numpy(),
                                 call.sw.cpu().numpy(), None, call.stride, call.pad, prod.as_tuple(), acc.as_tuple(),
                                 order, 16, ms, ns)
    else:
        lba.lba_gemm(call.x, call.w, call.sx, call.sw, None, prod, acc, order, 16, out=out)
        want = orc.gemm_points(call.x.cpu().numpy(), call.w.cpu().numpy(), call.sx.cpu().numpy(),
                               call.sw.cpu().numpy(), None, prod.as_tuple(), acc.as_tuple(), order, 16, ms, ns)
    _assert_points_equal(out, ms, ns, want, f"{call.name} {call.kind} {m}x{n}x{k} order {order}")
    return out


def _resnet(arch, batch, config, tiles, wa_format="e4m3"):
    prod, acc = code_domain_formats(7, 4) if wa_format == "e4m3" else m4e3_input_formats(7, 4)

    def conv_fn(x, w, sx, sw, stride, pad):
        return lba.lba_conv2d(x, w, sx, sw, None, stride, pad, prod, acc, CHK, 16)

    def gemm_fn(a, b, sa, sb):
        return lba.lba_gemm(a, b, sa, sb, None, prod, acc, CHK, 16)

    calls, logits = workloads.build_resnet_calls(arch, batch, config, DEV, conv_fn, gemm_fn, wa_format=wa_format)
    assert torch.isfinite(logits).all()
    for i, call in enumerate(calls):
        _check_call(call, prod, acc, CHK, tiles, 1000 * config + 10 * i)
    # the sequential order on a subset: the stem, one 3x3 per stage and the final linear layer
    picks = [calls[0]] + [c for c in calls if c.name.endswith(".1.conv2")] + [calls[-1]]
    for i, call in enumerate(picks):
        _check_call(call, prod, acc, SEQ, max(8, tiles // 4), 1000 * config + 500 + i)
    return calls


def test_config2_resnet18_batch32_every_conv_and_fc():
    calls = _resnet("resnet18", 32, 2, tiles=64)
    assert len(calls) == 21
    assert sum(c.macs for c in calls) == 58050347008          # 1.81 GMAC per image, batch 32
    torch.cuda.empty_cache()


def test_resnet18_batch32_in_the_papers_own_wa_format():
    # the forward regime of the paper's FP8 runs (Sec. 3.1, Table 3): weights and activations in the M4E3 byte format
    # with one power-of-two flex-bias per tensor, M7E4 product and accumulator formats; products carry ten
    # significant bits here, so Q_prod really cuts the mantissa
    calls = _resnet("resnet18", 32, 2, tiles=32, wa_format="m4e3")
    assert len(calls) == 21
    prod, _ = m4e3_input_formats(7, 4)
    assert "pq=cut" in lba.describe_plan(*calls[3].gemm_shape, prod, _, CHK, 16, is_conv=True)
    torch.cuda.empty_cache()


def test_config3_resnet50_batch64_every_conv_and_fc():
    calls = _resnet("resnet50", 64, 3, tiles=32)
    assert len(calls) == 54
    assert max(c.gemm_shape[2] for c in calls) == 4608
    torch.cuda.empty_cache()


def test_config4_bert_base_linears_with_outlier_channels():
    prod, acc = code_domain_formats(7, 4)
    calls = workloads.build_bert_calls(4096, 4, DEV)
    assert [c.gemm_shape for c in calls] == [(4096, 768, 768)] * 4 + [(4096, 3072, 768), (4096, 768, 3072)]
    for i, call in enumerate(calls):
        for order in (CHK, SEQ):
            _check_call(call, prod, acc, order, 64, 4000 + 10 * i + order)
    # the outlier channels make most products small: the Q_prod flush must be active here
    a = synth.e4m3_decode(calls[0].x[:64].cpu()).numpy().astype(np.float64)
    b = synth.e4m3_decode(calls[0].w[:64].cpu()).numpy().astype(np.float64)
    p = np.abs(a[:, None, :] * b[None, :, :])
    assert ((p > 0) & (p < r_uf(prod))).mean() > 0.01


SWEEP = [(m, e, r) for e in (4, 5, 6) for m in range(4, 11) for r in (0, 1)]


def test_config5_accumulator_format_sweep_8192():
    # M = N = K = 8192, N(0,1) operands; mantissa 4..10 x exponent 4..6 x {floor, nearest-even}; Q_prod follows
    # Q_acc; the same 256 seeded 16x16 output tiles are checked at every point of the sweep
    A, sa, B, sb = synth.gemm_case(8192, 8192, 8192, config=5)
    An, Bn, san, sbn = A.numpy(), B.numpy(), sa.numpy(), sb.numpy()
    A, B, sa, sb = A.to(DEV), B.to(DEV), sa.to(DEV), sb.to(DEV)
    out = torch.empty((8192, 8192), dtype=torch.float32, device=DEV)
    ms, ns = synth.sample_tiles(8192, 8192, 256, 16, 5005)
    plans = set()
    for (m, e, r) in SWEEP:
        prod, acc = code_domain_formats(m, e, rounding=r)
        lba.lba_gemm(A, B, sa, sb, None, prod, acc, CHK, 16, out=out)
        want = orc.gemm_points(An, Bn, san, sbn, None, prod.as_tuple(), acc.as_tuple(), CHK, 16, ms, ns)
        _assert_points_equal(out, ms, ns, want, f"sweep M{m}E{e} rounding {r}")
        plans.add(lba.describe_plan(8192, 8192, 8192, prod, acc, CHK, 16).split("q=")[1].split()[0])
    assert {"floor_fast", "floor_full", "rne_full"} <= plans


def _row_col_blocks(M, N, blocks, seed):
    g = torch.Generator().manual_seed(seed)
    m0 = torch.randint(0, M // 16, (blocks,), generator=g) * 16
    n0 = torch.randint(0, N // 16, (blocks,), generator=g) * 16
    return [(int(a), int(b)) for a, b in zip(m0, n0)]


def test_bert_ffn_shape_ste_masks_and_fixed_point_at_full_size():
    # the shape bench.py times for the mask re-computation and the fixed-point accumulator (BERT-base FFN-in,
    # 4096 x 3072 x 768): seeded 16 x 16 output blocks against the oracle run on the same rows of A and B
    M, N, K = 4096, 3072, 768
    A, sa, B, sb = synth.gemm_case(M, N, K, config=5)
    An, Bn = A.numpy(), B.numpy()
    Ad, Bd, sad, sbd = A.to(DEV), B.to(DEV), sa.to(DEV), sb.to(DEV)
    prod, acc = code_domain_formats(7, 4)
    blocks = _row_col_blocks(M, N, 24, 99)
    for order, chunk in ((CHK, 16), (SEQ, 1)):
        for kind, okind, e1, e2 in ((lba.STE_OF, orc.STE_OF, 0.0, 0.0), (lba.STE_DIFF, orc.STE_DIFF, 2.0 ** -20, 0.25)):
            g1, g2 = lba.lba_gemm_ste_mask(Ad, Bd, prod, acc, order, chunk, kind, e1, e2)
            zeros = 0
            for m0, n0 in blocks:
                w1, w2 = orc.gemm_ste_mask(An[m0:m0 + 16], Bn[n0:n0 + 16], prod.as_tuple(), acc.as_tuple(), order, chunk,
                                           okind, e1, e2)
                got1 = g1[m0:m0 + 16, :, n0:n0 + 16].cpu().numpy().view(np.uint32)
                assert (got1 == w1).all(), f"mask1 order {order} kind {kind} block ({m0}, {n0})"
                if w2 is not None:
                    got2 = g2[m0:m0 + 16, :, n0:n0 + 16].cpu().numpy().view(np.uint32)
                    assert (got2 == w2).all(), f"mask2 order {order} kind {kind} block ({m0}, {n0})"
                zeros += int(w1.size * 32 - np.unpackbits(w1.view(np.uint8)).sum())
            assert kind == lba.STE_OF or zeros > 0          # swamped steps exist on Gaussian data
            del g1, g2
    last = lba.lba_gemm_last_overflow(Ad, Bd, prod, acc)
    for m0, n0 in blocks:
        want = orc.gemm_last_overflow(An[m0:m0 + 16], Bn[n0:n0 + 16], prod.as_tuple(), acc.as_tuple())
        assert (last[m0:m0 + 16, n0:n0 + 16].cpu().numpy() == want).all()
    # fixed-point accumulators in the formats of the benchmark's fixed-point workload
    out = torch.empty((M, N), dtype=torch.float32, device=DEV)
    ms, ns = synth.sample_tiles(M, N, 64, 16, 4242)
    for wrap in (False, True):
        pf, af = fixed_point_format(12, -7, wrap), fixed_point_format(12, -9, wrap)
        for order in (CHK, SEQ):
            lba.lba_gemm(Ad, Bd, sad, sbd, None, pf, af, order, 16, out=out)
            want = orc.gemm_points(An, Bn, sa.numpy(), sb.numpy(), None, pf.as_tuple(), af.as_tuple(), order, 16, ms, ns)
            _assert_points_equal(out, ms, ns, want, f"fixed point wrap={wrap} order {order}")
    torch.cuda.empty_cache()
