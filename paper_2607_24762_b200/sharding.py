"""Host-side helpers for running the softmax on several GPUs of one node.

Rows are independent, so the path shards by contiguous row blocks with no exchange of data: each
rank owns rows [row_shard(rows, rank, world)) of a tensor, or, as in the benchmark, a whole
per-GPU copy of the workload (weak scaling). The only communication is the reduction of the timing:
a job is as slow as its slowest rank.
"""
from __future__ import annotations


def row_shard(rows: int, rank: int, world: int) -> tuple[int, int]:
    """Rows [lo, hi) of rank `rank` when `rows` rows are split over `world` ranks.

    Contiguous, disjoint, covering; sizes differ by at most one (the first rows % world ranks get
    the extra row).
    """
    if world < 1 or not (0 <= rank < world) or rows < 0:
        raise ValueError("bad shard request")
    base, extra = divmod(rows, world)
    lo = rank * base + min(rank, extra)
    return lo, lo + base + (1 if rank < extra else 0)


def max_over_ranks(value: float, device=None) -> float:
    """MAX all-reduce of a per-rank scalar (a step time); the identity without a process group."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device if device is not None else "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def aggregate_throughput(units_per_rank: float, seconds_max: float, world: int) -> float:
    """Whole-job throughput when every rank processes `units_per_rank` units (weak scaling)."""
    return world * units_per_rank / seconds_max
