"""Exhaustive two-step chains on the GPU: every ordered pair of finite E4M3 codes as (x_0, x_1) against every ordered
pair as (w_0, w_1), 64516^2 = 4.2e9 chains of K = 2, M7E4, floor, sequential order.

Opt-in (set LBA_EXHAUSTIVE=1; about a quarter of an hour): the C++ oracle takes hours for this many chains, so the full
comparison is against the 64-bit integer coding of Eq. 2 / Eq. 4 (tests/helpers/int_coding.py, itself pinned against the
oracle over all code pairs and a covering set of running sums in the CPU suite), block of rows by block of rows so that
neither the 16.6 GB of outputs nor the reference is ever held at once; a seeded sample of two million chains is checked
against the oracle itself.  Needs a B200."""
import os

import numpy as np
import pytest
import torch

from oracle import lba_oracle as orc
from paper_2401_14110_b200 import binding as lba
from paper_2401_14110_b200 import code_domain_formats, ORDER_SEQUENTIAL as SEQ
from helpers import int_coding as ic

pytestmark = [pytest.mark.gpu, pytest.mark.skipif(os.environ.get("LBA_EXHAUSTIVE") != "1",
                                                  reason="opt-in: set LBA_EXHAUSTIVE=1 (4.2e9 chains)")]

DEV = "cuda:0"
FINITE = np.array([c for c in range(256) if (c & 0x7F) != 0x7F], dtype=np.uint8)


@pytest.mark.parametrize("rounding", [0, 1])
def test_every_two_step_chain_m7e4(rounding):
    prod, acc = code_domain_formats(7, 4, rounding)
    n = len(FINITE)
    pairs = np.stack([np.repeat(FINITE, n), np.tile(FINITE, n)], axis=1)          # [64516][2]: (c_0, c_1)
    U = 32
    val = np.zeros(256, dtype=np.int64)
    for c in FINITE:
        val[c] = ic.e4m3_int(int(c), U // 2)
    w0, w1 = val[pairs[:, 0]][None, :], val[pairs[:, 1]][None, :]
    B = torch.from_numpy(pairs).to(DEV)
    one = torch.ones(1, device=DEV)
    rng = np.random.default_rng(2024)
    rows_per_block = 256
    out = torch.empty((rows_per_block, n * n), dtype=torch.float32, device=DEV)
    pf, af = prod.as_tuple(), acc.as_tuple()
    sample_m, sample_n, sample_got = [], [], []
    for r0 in range(0, n * n, rows_per_block):
        rows = pairs[r0:r0 + rows_per_block]
        o = out[:len(rows)]
        lba.lba_gemm(torch.from_numpy(rows).to(DEV), B, one, one, None, prod, acc, SEQ, 1, out=o)
        got = o.cpu().numpy()
        x0, x1 = val[rows[:, 0]][:, None], val[rows[:, 1]][:, None]
        s1 = ic.fmaq_int(pf, af, x0, w0, 0, U)                                    # Eq. 8-9, two steps
        s2 = ic.fmaq_int(pf, af, x1, w1, s1, U)
        want = np.ldexp(s2.astype(np.float64), -U).astype(np.float32)
        bad = np.argwhere(got.view(np.uint32) != want.view(np.uint32))
        assert bad.size == 0, (f"rounding {rounding}: x codes {rows[bad[0][0]]}, w codes {pairs[bad[0][1]]}: gpu "
                               f"{got[tuple(bad[0])]!r}, integer coding {want[tuple(bad[0])]!r}")
        k = rng.integers(0, got.size, 8000)
        sample_m.append(r0 + k // (n * n))
        sample_n.append(k % (n * n))
        sample_got.append(got.reshape(-1)[k])
    ms, ns = np.concatenate(sample_m), np.concatenate(sample_n)
    ref = orc.gemm_points(pairs, pairs, 1.0, 1.0, None, pf, af, SEQ, 1, ms, ns)
    assert np.array_equal(ref.view(np.uint32), np.concatenate(sample_got).view(np.uint32))
