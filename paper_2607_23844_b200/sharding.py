"""Multi-GPU plumbing: how independent token groups are spread over ranks, and rank aggregation.

The path shards without any data exchange: a group (a batch element, a frame, a patch) is matched,
selected, gathered and restored on its own, so each rank owns a contiguous range of groups and the
only cross-rank traffic is the timing barrier and a max / sum of scalars.  Works with the ``nccl``
backend on GPUs and with ``gloo`` on CPU (used by the tests).
"""
from __future__ import annotations

import os

import torch
import torch.distributed as dist


def env_rank_world() -> tuple[int, int, int]:
    """(rank, local_rank, world_size) from the torchrun environment; (0, 0, 1) when absent."""
    return (int(os.environ.get("RANK", 0)), int(os.environ.get("LOCAL_RANK", 0)),
            int(os.environ.get("WORLD_SIZE", 1)))


def group_range(n_groups: int, rank: int, world: int) -> tuple[int, int]:
    """Contiguous, balanced partition of ``n_groups`` independent groups: rank r owns [lo, hi)."""
    if not (0 <= rank < world) or n_groups < 0:
        raise ValueError("bad rank / world / n_groups")
    base, extra = divmod(n_groups, world)
    lo = rank * base + min(rank, extra)
    return lo, lo + base + (1 if rank < extra else 0)


def init(backend: str | None = None) -> tuple[int, int, int]:
    """Initialises torch.distributed from the environment when world_size > 1."""
    rank, local_rank, world = env_rank_world()
    if world > 1 and not dist.is_initialized():
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        if backend is None:
            backend = "nccl" if torch.cuda.is_available() else "gloo"
        kwargs = {}
        if backend == "nccl":
            kwargs["device_id"] = torch.device("cuda", local_rank)
        dist.init_process_group(backend=backend, rank=rank, world_size=world, **kwargs)
    return rank, local_rank, world


def _reduce(value: float, op, device) -> float:
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([value], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=op)
    return float(t.item())


def max_over_ranks(value: float, device="cpu") -> float:
    return _reduce(value, dist.ReduceOp.MAX, device)


def sum_over_ranks(value: float, device="cpu") -> float:
    return _reduce(value, dist.ReduceOp.SUM, device)


def barrier() -> None:
    if dist.is_available() and dist.is_initialized() and dist.get_world_size() > 1:
        dist.barrier()


def finalize() -> None:
    if dist.is_available() and dist.is_initialized():
        dist.destroy_process_group()
