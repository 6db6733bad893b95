"""Rank plumbing for data-parallel use of the DDTS library: (sequence, head) units are independent,
so ranks take disjoint shares of the sequences and nothing crosses ranks on the data path.  Only
timing (max over ranks) and bookkeeping (sums) are reduced, over NCCL on GPUs or gloo on CPU."""
from __future__ import annotations

import os
from typing import Optional, Tuple


def env_rank() -> Tuple[int, int, int]:
    """(rank, world_size, local_rank) from the torchrun environment; (0, 1, 0) outside it."""
    return (int(os.environ.get("RANK", "0")), int(os.environ.get("WORLD_SIZE", "1")),
            int(os.environ.get("LOCAL_RANK", "0")))


def init(backend: str, device=None) -> Tuple[int, int]:
    """Initialises the default process group when WORLD_SIZE > 1; returns (rank, world)."""
    import torch.distributed as dist
    rank, world, _ = env_rank()
    if world > 1 and not dist.is_initialized():
        kw = {"device_id": device} if (backend == "nccl" and device is not None) else {}
        dist.init_process_group(backend, **kw)
    return rank, world


def shard_units(n_units: int, rank: int, world: int) -> range:
    """Contiguous, near-equal share of ``n_units`` independent units for ``rank`` (sizes differ by
    at most one; earlier ranks take the larger shares)."""
    base, extra = divmod(n_units, world)
    lo = rank * base + min(rank, extra)
    return range(lo, lo + base + (1 if rank < extra else 0))


def _reduce(value: float, op_name: str, device=None) -> float:
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([value], dtype=torch.float64, device=device if device is not None else "cpu")
    dist.all_reduce(t, op=getattr(dist.ReduceOp, op_name))
    return float(t.item())


def max_over_ranks(value: float, device=None) -> float:
    return _reduce(value, "MAX", device)


def sum_over_ranks(value: float, device=None) -> float:
    return _reduce(value, "SUM", device)


def barrier() -> None:
    import torch.distributed as dist
    if dist.is_available() and dist.is_initialized() and dist.get_world_size() > 1:
        dist.barrier()


def aggregate_throughput(units_this_rank: float, seconds_this_rank: float, device=None) -> float:
    """Whole-job rate: all ranks' units over the slowest rank's time."""
    return sum_over_ranks(units_this_rank, device) / max_over_ranks(seconds_this_rank, device)
