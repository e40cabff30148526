"""Prefill of one long sequence cut along the sequence over several GPUs (one process per GPU).

Every rank holds one contiguous stretch of the tokens.  Between stretches the layer carries only the cumulative
sums S = sum phi(k) v^T and z = sum phi(k) and the last W-1 values of v (Sec. 4.1: group-level cumulative sums), so:

  1. every rank computes the sums of its own stretch            (la_segment_state: K and V are read once),
  2. one all-gather exchanges them (B*H*(d*d+d)*4 bytes per rank, 2.1 MB at H = 32, d = 128) together with each
     rank's last W-1 values of v,
  3. every rank adds up the sums of the ranks before it         (la_state_prefix),
  4. and runs the ordinary prefill on its stretch from that state (la_prefill with init_state = 1).

The arithmetic of steps 1, 3 and 4 runs in the library's kernels; this module only slices, gathers and marshals.
`ops` and `comm` are injected so that the same host logic can be driven without GPUs (gloo ranks with a CPU
stand-in for the kernels) and on one GPU (all ranks in one process, one after the other).
"""
from __future__ import annotations

from dataclasses import dataclass

import torch


def token_shard(T: int, rank: int, world: int, multiple: int = 128) -> tuple[int, int]:
    """[lo, hi) of `rank`: stretches of equal length rounded up to `multiple` tokens, the last one shorter (or empty)."""
    per = -(-T // world)
    per = -(-per // multiple) * multiple
    lo = min(T, rank * per)
    return lo, min(T, lo + per)


@dataclass
class Partial:
    """What a rank contributes to the exchange: the sums of its stretch and its last W-1 values of v."""
    dS: torch.Tensor       # [B, H, d, d] fp32
    dz: torch.Tensor       # [B, H, d] fp32
    tail: torch.Tensor     # [B, H, W-1, d] io type: the last min(T_loc, W-1) values of v, right-aligned
    count: int             # tokens of the stretch


class BindingOps:
    """The library's kernels behind the three compute steps."""

    def __init__(self, ctx):
        self.ctx = ctx
        self.W = ctx.W

    def segment_state(self, k, v):
        return self.ctx.la_segment_state(k, v)

    def state_prefix(self, dS_parts, dz_parts, count, S_base, z_base):
        return self.ctx.la_state_prefix(dS_parts, dz_parts, count, S_base, z_base)

    def prefill_from(self, q, k, v, conv_w, S, z, win, pos, have_state):
        from . import binding
        st = binding.State(S, z, win, pos)
        o = self.ctx.la_prefill(q, k, v, conv_w, st, init_state=have_state)
        return o


class TorchDistComm:
    """All-gather over torch.distributed (NCCL on GPUs, gloo on CPU)."""

    def __init__(self, group=None):
        import torch.distributed as td
        self.td, self.group = td, group

    def all_gather(self, x: torch.Tensor) -> torch.Tensor:
        world = self.td.get_world_size(self.group)
        parts = [torch.empty_like(x) for _ in range(world)]
        self.td.all_gather(parts, x.contiguous(), group=self.group)
        return torch.stack(parts)


def local_partial(ops, k_loc, v_loc, W: int) -> Partial:
    """Step 1 on one rank.  An empty stretch contributes zeros."""
    B, H, T, d = k_loc.shape
    tail = torch.zeros(B, H, W - 1, d, dtype=v_loc.dtype, device=v_loc.device)
    if T == 0:
        return Partial(torch.zeros(B, H, d, d, dtype=torch.float32, device=k_loc.device),
                       torch.zeros(B, H, d, dtype=torch.float32, device=k_loc.device), tail, 0)
    dS, dz = ops.segment_state(k_loc.contiguous(), v_loc.contiguous())
    n = min(T, W - 1)
    if n:
        tail[:, :, W - 1 - n:] = v_loc[:, :, T - n:]
    return Partial(dS, dz, tail, T)


def window_before(rank: int, tails: torch.Tensor, counts: list[int], win0: torch.Tensor | None) -> torch.Tensor:
    """The last W-1 values of v before `rank`'s stretch: the caller's window, then the tails of the ranks before."""
    W1 = tails.shape[3]
    seq = [win0 if win0 is not None else torch.zeros_like(tails[0])]
    for r in range(rank):
        n = min(counts[r], W1)
        if n:
            seq.append(tails[r][:, :, W1 - n:])
    return torch.cat(seq, dim=2)[:, :, -W1:].contiguous() if W1 else tails[0]


def finish_rank(ops, rank: int, q_loc, k_loc, v_loc, conv_w, dS_all, dz_all, tails, counts, state0):
    """Steps 3 and 4 on one rank.  Returns (o_loc, final S, final z, final window, final pos): the final state is the
    same on every rank (the caller's state plus the sums of all stretches)."""
    world = dS_all.shape[0]
    S0 = z0 = win0 = pos0 = None
    if state0 is not None:
        S0, z0, win0, pos0 = state0
    B = dS_all.shape[1]
    before = sum(counts[:rank])
    pos_base = pos0.clone() if pos0 is not None else torch.zeros(B, dtype=torch.int64, device=dS_all.device)
    pos_start = pos_base + before                     # the prefill advances this tensor in place
    o = None
    if q_loc.shape[2] > 0:
        S, z = ops.state_prefix(dS_all, dz_all, rank, S0, z0)
        win = window_before(rank, tails, counts, win0)
        o = ops.prefill_from(q_loc.contiguous(), k_loc.contiguous(), v_loc.contiguous(), conv_w, S, z, win, pos_start,
                             state0 is not None or before > 0)
    S_fin, z_fin = ops.state_prefix(dS_all, dz_all, world, S0, z0)
    win_fin = window_before(world, tails, counts, win0)
    pos_fin = pos_base + sum(counts)
    return o, S_fin, z_fin, win_fin, pos_fin


def sequence_parallel_prefill(ops, comm, rank: int, q_loc, k_loc, v_loc, conv_w, W: int, state0=None):
    """The whole exchange on one rank of a running process group.  q_loc, k_loc, v_loc: this rank's stretch
    [B, H, T_loc, d] (see token_shard); state0: (S, z, win, pos) to continue from, identical on all ranks, or None."""
    part = local_partial(ops, k_loc, v_loc, W)
    dS_all = comm.all_gather(part.dS)
    dz_all = comm.all_gather(part.dz)
    tails = comm.all_gather(part.tail)
    counts = comm.all_gather(torch.tensor([part.count], dtype=torch.int64, device=part.dS.device)).view(-1).tolist()
    return finish_rank(ops, rank, q_loc, k_loc, v_loc, conv_w, dS_all, dz_all, tails, counts, state0)
