"""torch.distributed plumbing for multi-process runs (one process per GPU).

The operator has no cross-GPU exchange: (batch, head) pairs are independent, so ranks run
independent replicas and the only collectives are the benchmark's own barrier and the
max / sum over ranks of its timings and unit counts.
"""
from __future__ import annotations

import os

import torch
import torch.distributed as td


def init_from_env(backend: str):
    """(rank, world_size, local_rank) from torchrun's environment; no process group when WORLD_SIZE is 1."""
    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if world > 1 and not td.is_initialized():
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        os.environ.setdefault("MASTER_PORT", "29500")
        if backend == "nccl":
            torch.cuda.set_device(local)
        td.init_process_group(backend=backend, rank=rank, world_size=world)
    return rank, world, local


def _active() -> bool:
    return td.is_available() and td.is_initialized() and td.get_world_size() > 1


def _reduce(x: float, op) -> float:
    if not _active():
        return float(x)
    dev = "cuda" if td.get_backend() == "nccl" else "cpu"
    t = torch.tensor([x], dtype=torch.float64, device=dev)
    td.all_reduce(t, op=op)
    return float(t.item())


def max_over_ranks(x: float) -> float:
    return _reduce(x, td.ReduceOp.MAX)


def sum_over_ranks(x: float) -> float:
    return _reduce(x, td.ReduceOp.SUM)


def barrier() -> None:
    if _active():
        td.barrier()


def shard_range(total: int, rank: int, world: int):
    """Contiguous, balanced share [lo, hi) of `total` independent units for `rank` (first ranks get the extras)."""
    base, extra = divmod(total, world)
    lo = rank * base + min(rank, extra)
    return lo, lo + base + (1 if rank < extra else 0)


def shutdown() -> None:
    if td.is_available() and td.is_initialized():
        td.destroy_process_group()
