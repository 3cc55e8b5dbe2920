"""Data-parallel sharding of the LBA contraction across GPUs (one process per GPU).

Every output element is an independent accumulation chain, so the rows of A (the batch / token / output-pixel
dimension) are split across ranks, the weights are replicated, and each rank's output rows stay with it: no
collective is needed on the data path (the paper's own multi-GPU runs split the mini-batch the same way,
App. C.1).  K is never split: the accumulation order is part of the result (App. D).  The only communication
is control: a barrier and the reduction of per-rank timings.
"""
from typing import List, Tuple


def shard_rows(total: int, world: int, rank: int) -> Tuple[int, int]:
    """[begin, end) of the rows rank ``rank`` owns: contiguous, sizes differ by at most one, earlier ranks
    take the larger shards."""
    if world < 1 or not (0 <= rank < world) or total < 0:
        raise ValueError("bad shard request")
    base, extra = divmod(total, world)
    begin = rank * base + min(rank, extra)
    return begin, begin + base + (1 if rank < extra else 0)


def shard_sizes(total: int, world: int) -> List[int]:
    return [shard_rows(total, world, r)[1] - shard_rows(total, world, r)[0] for r in range(world)]


def max_over_ranks(value: float, dist=None, device=None) -> float:
    """The slowest rank's value (a job is as slow as its slowest GPU).  ``dist`` is torch.distributed or None."""
    if dist is None or not dist.is_initialized() or dist.get_world_size() == 1:
        return float(value)
    import torch
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_rate(units_per_rank: float, world: int, seconds: float) -> float:
    """Aggregate throughput when every rank processed ``units_per_rank`` units in ``seconds`` (max over ranks)."""
    return units_per_rank * world / seconds
