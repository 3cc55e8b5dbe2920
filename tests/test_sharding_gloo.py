"""The multi-GPU path on CPU: two gloo ranks shard the rows of one contraction, each computes its shard, and the
gathered result equals the unsharded one bit for bit (rows are independent chains; K is never split).  The
per-shard arithmetic here is the CPU oracle standing in for the GPU kernel: what is under test is the host
logic (row partition, timing reduction, aggregate rate), which is what bench.py uses with N > 1."""
import os
import socket
import sys

import numpy as np
import pytest
import torch
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2401_14110_b200 import sharding, synth, code_domain_formats, ORDER_CHUNKED  # noqa: E402


def test_shard_rows_partition_exactly():
    for total in (0, 1, 7, 64, 1568, 100352):
        for world in (1, 2, 3, 8):
            spans = [sharding.shard_rows(total, world, r) for r in range(world)]
            assert spans[0][0] == 0 and spans[-1][1] == total
            assert all(spans[i][1] == spans[i + 1][0] for i in range(world - 1))
            sizes = sharding.shard_sizes(total, world)
            assert sum(sizes) == total and max(sizes) - min(sizes) <= 1
    with pytest.raises(ValueError):
        sharding.shard_rows(10, 2, 2)
    assert sharding.whole_job_rate(100.0, 4, 2.0) == 200.0
    assert sharding.max_over_ranks(3.5) == 3.5


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    return port


def _worker(rank, world, port, M, N, K, out_path):
    import torch.distributed as dist
    from oracle import lba_oracle as orc
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        prod, acc = code_domain_formats(7, 4)
        A, sa, B, sb = synth.gemm_case(M, N, K, config=90)        # same seeded inputs on every rank
        lo, hi = sharding.shard_rows(M, world, rank)
        mine = orc.gemm(A[lo:hi].numpy(), B.numpy(), sa.numpy(), sb.numpy(), None, prod.as_tuple(), acc.as_tuple(),
                        ORDER_CHUNKED, 16, nthreads=1)
        # control traffic only: the slowest rank's time; the output shards stay where they are
        slowest = sharding.max_over_ranks(1.0 + rank, dist)
        assert slowest == float(world)
        # for the check alone, collect the shards on rank 0
        parts = [None] * world
        dist.all_gather_object(parts, (lo, hi, mine.tobytes()))
        if rank == 0:
            full = np.empty((M, N), dtype=np.float32)
            for lo_r, hi_r, raw in parts:
                full[lo_r:hi_r] = np.frombuffer(raw, dtype=np.float32).reshape(hi_r - lo_r, N)
            np.save(out_path, full)
        dist.barrier()
    finally:
        dist.destroy_process_group()


def test_two_ranks_row_sharded_equals_unsharded(tmp_path):
    from oracle import lba_oracle as orc
    M, N, K = 37, 24, 96                     # an odd row count: the shards differ in size
    out_path = str(tmp_path / "gathered.npy")
    mp.spawn(_worker, args=(2, _free_port(), M, N, K, out_path), nprocs=2, join=True)
    prod, acc = code_domain_formats(7, 4)
    A, sa, B, sb = synth.gemm_case(M, N, K, config=90)
    want = orc.gemm(A.numpy(), B.numpy(), sa.numpy(), sb.numpy(), None, prod.as_tuple(), acc.as_tuple(),
                    ORDER_CHUNKED, 16)
    got = np.load(out_path)
    assert np.array_equal(got.view(np.uint32), want.view(np.uint32))
