"""Token sharding across ranks.  Token rows are independent in both kernels of the path, so a
batch is split by rows, map and weights are replicated, and no collective touches the data path;
the only cross-rank exchange is the reduction of timings / statuses."""
from __future__ import annotations


def token_shard(M: int, rank: int, world: int) -> tuple[int, int]:
    """(first row, row count) of `rank`'s contiguous share of M token rows; shares differ by at most one."""
    if world <= 0 or not (0 <= rank < world) or M < 0:
        raise ValueError("bad shard arguments")
    base, extra = divmod(M, world)
    start = rank * base + min(rank, extra)
    return start, base + (1 if rank < extra else 0)


def max_over_ranks(value: float, group=None) -> float:
    """Largest value over all ranks (how step times of a multi-GPU run are combined)."""
    import torch
    import torch.distributed as dist
    if not dist.is_available() or not dist.is_initialized() or dist.get_world_size(group) == 1:
        return float(value)
    dev = "cuda" if dist.get_backend(group) == "nccl" else "cpu"
    t = torch.tensor([float(value)], dtype=torch.float64, device=dev)
    dist.all_reduce(t, op=dist.ReduceOp.MAX, group=group)
    return float(t.item())
