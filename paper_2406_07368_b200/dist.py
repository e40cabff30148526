"""Multi-process plumbing for replicated runs: one process per GPU, no data-path collective.

Every (sequence, head) unit of the layer is independent, so ranks only meet to line up the
timed region (a barrier) and to agree on the slowest rank's time (a MAX all-reduce).
"""
from __future__ import annotations

import os
import socket
import subprocess
import time

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


def free_port() -> int:
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def launch_local_ranks(cmd: list[str], world: int, timeout: float | None = None, env: dict | None = None) -> int:
    """Starts `world` copies of `cmd` on this node, one per rank (RANK = LOCAL_RANK = 0 .. world-1, WORLD_SIZE,
    MASTER_ADDR = 127.0.0.1 and a free MASTER_PORT in the environment), and waits for them.  All ranks inherit this
    process's stdout and stderr.  Returns 0 if every rank exited 0, otherwise the first non-zero exit code (after
    ending the ranks that were still running: only processes started here, by their own handles)."""
    base = dict(os.environ if env is None else env)
    base.update(WORLD_SIZE=str(world), MASTER_ADDR="127.0.0.1", MASTER_PORT=str(free_port()))
    procs = []
    for r in range(world):
        procs.append(subprocess.Popen(cmd, env=dict(base, RANK=str(r), LOCAL_RANK=str(r))))
    deadline = None if timeout is None else time.time() + timeout
    rc = 0
    pending = list(procs)
    while pending and rc == 0:
        for p in list(pending):
            code = p.poll()
            if code is not None:
                pending.remove(p)
                if code != 0:
                    rc = code
        if deadline is not None and time.time() > deadline:
            rc = 124
        if pending and rc == 0:
            time.sleep(0.05)
    for p in pending:                                   # a rank failed or time ran out: end the others
        p.terminate()
    for p in pending:
        try:
            p.wait(timeout=10)
        except subprocess.TimeoutExpired:
            p.kill()
    return rc
