"""Exhaustive two-step chains on the GPU: every ordered pair of finite E4M3 codes as (x_0, x_1) against every ordered
pair as (w_0, w_1), 64516^2 = 4.2e9 chains of K = 2, M7E4, sequential order, floor and nearest-even.

The GPU result is compared bit for bit with the C++ oracle on every one of the chains, block of rows by block of rows,
so that neither the 16.6 GB of outputs nor the reference is ever held at once: about 45 s per rounding with 16 host cores
(the oracle's share is 4.2e9 chains at its 0.35 GMAC/s).  LBA_SKIP_EXHAUSTIVE=1 skips it.  K = 3 would be 2.7e14 chains:
longer chains are covered by the covering-set test of the CPU suite and by seeded samples.  Needs a B200."""
import os

import numpy as np
import pytest
import torch

from oracle import lba_oracle as orc
from paper_2401_14110_b200 import binding as lba
from paper_2401_14110_b200 import code_domain_formats, ORDER_SEQUENTIAL as SEQ

pytestmark = [pytest.mark.gpu, pytest.mark.skipif(os.environ.get("LBA_SKIP_EXHAUSTIVE") == "1",
                                                  reason="LBA_SKIP_EXHAUSTIVE=1 (4.2e9 chains per rounding)")]

DEV = "cuda:0"
FINITE = np.array([c for c in range(256) if (c & 0x7F) != 0x7F], dtype=np.uint8)


@pytest.mark.parametrize("rounding", [0, 1])
def test_every_two_step_chain_m7e4(rounding):
    prod, acc = code_domain_formats(7, 4, rounding)
    n = len(FINITE)
    pairs = np.stack([np.repeat(FINITE, n), np.tile(FINITE, n)], axis=1)          # [64516][2]: (c_0, c_1)
    B = torch.from_numpy(pairs).to(DEV)
    one = torch.ones(1, device=DEV)
    rows_per_block = 1024
    out = torch.empty((rows_per_block, n * n), dtype=torch.float32, device=DEV)
    pf, af = prod.as_tuple(), acc.as_tuple()
    saturated = 0
    for r0 in range(0, n * n, rows_per_block):
        rows = pairs[r0:r0 + rows_per_block]
        o = out[:len(rows)]
        lba.lba_gemm(torch.from_numpy(rows).to(DEV), B, one, one, None, prod, acc, SEQ, 1, out=o)
        got = o.cpu().numpy()
        want = orc.gemm(rows, pairs, 1.0, 1.0, None, pf, af, SEQ, 1)               # Eq. 8-9, two steps, every chain
        bad = np.argwhere(got.view(np.uint32) != want.view(np.uint32))
        assert bad.size == 0, (f"rounding {rounding}: x codes {rows[bad[0][0]]}, w codes {pairs[bad[0][1]]}: gpu "
                               f"{got[tuple(bad[0])]!r}, oracle {want[tuple(bad[0])]!r}")
        saturated += int((np.abs(want) == np.float32(1044480.0)).sum())
    assert saturated == 0          # two products cannot reach R_OF_acc = 1044480: the chains test rounding and flushes
