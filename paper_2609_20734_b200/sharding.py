"""Multi-GPU plumbing of the ODA decode path.  Requests are independent (the recall flag is per
request), so ranks take contiguous shards of the batch and no collective touches the data path;
the only exchanges are the reductions a benchmark or a server needs for its own bookkeeping."""
from __future__ import annotations


def request_shard(num_requests: int, rank: int, world: int) -> tuple[int, int]:
    """Contiguous [lo, hi) slice of the requests owned by `rank`; sizes differ by at most one."""
    base, rem = divmod(num_requests, world)
    lo = rank * base + min(rank, rem)
    return lo, lo + base + (1 if rank < rem else 0)


def max_over_ranks(value: float) -> float:
    """Slowest rank's time: what whole-job throughput is divided by."""
    import torch
    import torch.distributed as dist

    if not (dist.is_available() and dist.is_initialized()):
        return float(value)
    dev = "cuda" if dist.get_backend() == "nccl" else "cpu"
    t = torch.tensor([value], dtype=torch.float64, device=dev)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def sum_over_ranks(value: float) -> float:
    import torch
    import torch.distributed as dist

    if not (dist.is_available() and dist.is_initialized()):
        return float(value)
    dev = "cuda" if dist.get_backend() == "nccl" else "cpu"
    t = torch.tensor([value], dtype=torch.float64, device=dev)
    dist.all_reduce(t, op=dist.ReduceOp.SUM)
    return float(t.item())
