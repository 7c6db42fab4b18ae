"""Multi-GPU plumbing for the GEMM path: there is no data-path collective.

Rows of C = A x B are independent, so a product that is too tall for one GPU
is cut into row shards: rank r multiplies its rows of A by the whole of B and
owns the same rows of C.  Nothing is exchanged while computing; the process
group is only used to line the ranks up for timing (a barrier) and to take the
maximum of their device-side timings.
"""
from __future__ import annotations


def row_shard(M: int, rank: int, world: int):
    """Rows [begin, end) of an M-row product that rank ``rank`` of ``world``
    owns: contiguous, sizes differing by at most one, larger shards first."""
    if world < 1 or not (0 <= rank < world):
        raise ValueError("bad rank/world")
    base, extra = divmod(M, world)
    begin = rank * base + min(rank, extra)
    return begin, begin + base + (1 if rank < extra else 0)


def weak_scaling_rows(rows_per_gpu: int, world: int) -> int:
    """Total rows of the weak-scaling job: every GPU keeps ``rows_per_gpu``."""
    return rows_per_gpu * world


def max_over_ranks(value: float, device=None) -> float:
    """Maximum of a per-rank scalar over the default process group (identity
    when no group is initialised).  Used for the timing of multi-GPU runs."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()):
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def aggregate_throughput(units_per_rank: float, world: int, seconds_max: float) -> float:
    """Whole-job throughput: the units all ranks processed over the slowest rank's time."""
    return units_per_rank * world / seconds_max
