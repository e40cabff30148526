"""Multi-process plumbing for replicated runs: one process per GPU, no data-path collective.

Every (sequence, head) unit of the layer is independent, so ranks only meet to line up the
timed region (a barrier) and to agree on the slowest rank's time (a MAX all-reduce).
"""
from __future__ import annotations

import os

import torch
import torch.distributed as td


def rank_world() -> tuple[int, int]:
    return int(os.environ.get("RANK", 0)), int(os.environ.get("WORLD_SIZE", 1))


def init(world: int, backend: str = "nccl") -> None:
    if world > 1 and not td.is_initialized():
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        td.init_process_group(backend=backend)


def barrier(world: int) -> None:
    if world > 1:
        td.barrier()


def max_over_ranks(x: float, world: int, device="cpu") -> float:
    if world == 1:
        return float(x)
    t = torch.tensor([float(x)], dtype=torch.float64, device=device)
    td.all_reduce(t, op=td.ReduceOp.MAX)
    return float(t.item())


def shard(n_units: int, rank: int, world: int) -> tuple[int, int]:
    """Contiguous [lo, hi) slice of n independent units owned by `rank` (sizes differ by at most 1)."""
    base, extra = divmod(n_units, world)
    lo = rank * base + min(rank, extra)
    return lo, lo + base + (1 if rank < extra else 0)


def finish(world: int) -> None:
    if world > 1 and td.is_initialized():
        td.destroy_process_group()
