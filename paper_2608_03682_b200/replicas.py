"""Multi-GPU plumbing: the denoising loop shards by request and exchanges nothing while it runs
(the paper's data-parallel runners own their buffers, caches and solver state), so N GPUs are N
independent replicas.  The only collective is the timing reduction of the benchmark."""
from __future__ import annotations

from typing import Tuple

import torch


def shard_requests(n_requests: int, world: int, rank: int) -> Tuple[int, int]:
    """Contiguous [begin, end) range of requests owned by `rank`; sizes differ by at most one."""
    base, extra = divmod(n_requests, world)
    begin = rank * base + min(rank, extra)
    return begin, begin + base + (1 if rank < extra else 0)


def max_over_ranks(value: float, device: str = "cpu") -> float:
    """Maximum of `value` over all ranks (the job is as slow as its slowest replica)."""
    import torch.distributed as dist

    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def barrier() -> None:
    import torch.distributed as dist

    if dist.is_available() and dist.is_initialized() and dist.get_world_size() > 1:
        dist.barrier()
