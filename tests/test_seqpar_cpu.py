"""Sequence-parallel prefill, host side: two gloo ranks exchange the sums of their stretches.  The kernels are played
by the float64 oracle (a test may do that; the library itself never does), so what is checked is the slicing, the
order of the gathered parts, the prefix arithmetic over ranks, the window hand-over and the positions."""
import os
import sys

import numpy as np
import torch

from oracle import la_oracle as orc
from paper_2406_07368_b200 import dist as ladist, seqpar

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


class OracleOps:
    """CPU stand-in for the three compute steps, written with the oracle's functions."""

    def __init__(self, phi, eps):
        self.phi, self.eps = phi, eps

    def segment_state(self, k, v):
        B, H, T, d = k.shape
        z = np.zeros((B, H, T, d))
        _, st = orc.prefill_quadratic(z, k.numpy(), v.numpy(), np.zeros((H, d, 1)), self.phi, self.eps)
        return torch.from_numpy(st.S), torch.from_numpy(st.z)

    def state_prefix(self, dS_parts, dz_parts, count, S_base, z_base):
        S = dS_parts[:count].sum(0) + (S_base if S_base is not None else 0)
        z = dz_parts[:count].sum(0) + (z_base if z_base is not None else 0)
        return S, z

    def prefill_from(self, q, k, v, conv_w, S, z, win, pos, have_state):
        st = orc.State(S.numpy(), z.numpy(), win.numpy(), pos.numpy())
        o, _ = orc.prefill_quadratic(q.numpy(), k.numpy(), v.numpy(), conv_w.numpy(), self.phi, self.eps, st)
        return torch.from_numpy(o)


def _case(T, W, seed=0):
    rng = np.random.default_rng(seed)
    B, H, d = 2, 2, 4
    q, k, v = (torch.from_numpy(rng.standard_normal((B, H, T, d))) for _ in range(3))
    w = torch.from_numpy(rng.standard_normal((H, d, W)))
    return q, k, v, w


def test_token_shards_tile_the_sequence():
    for T in (1, 127, 128, 129, 1000, 32768):
        for world in (1, 2, 3, 8):
            cuts = [seqpar.token_shard(T, r, world) for r in range(world)]
            assert cuts[0][0] == 0 and cuts[-1][1] == T
            assert all(a[1] == b[0] for a, b in zip(cuts, cuts[1:]))
            assert all((hi - lo) % 128 == 0 or hi == T for lo, hi in cuts)


def _run_in_process(T, W, world, with_state, multiple):
    """All ranks in one process: phase 1 for every rank, the gather by stacking, phase 2 for every rank."""
    q, k, v, w = _case(T, W)
    ops = OracleOps("elu1", 0.0)
    state0 = ost0 = None
    if with_state:
        q0, k0, v0, _ = _case(9, W, seed=5)
        _, ost0 = orc.prefill_quadratic(q0.numpy(), k0.numpy(), v0.numpy(), w.numpy(), "elu1", 0.0)
        state0 = tuple(torch.from_numpy(x) for x in (ost0.S, ost0.z, ost0.win, ost0.pos))
    cuts = [seqpar.token_shard(T, r, world, multiple) for r in range(world)]
    parts = [seqpar.local_partial(ops, k[:, :, lo:hi], v[:, :, lo:hi], W) for lo, hi in cuts]
    dS_all, dz_all = torch.stack([p.dS for p in parts]), torch.stack([p.dz for p in parts])
    tails, counts = torch.stack([p.tail for p in parts]), [p.count for p in parts]
    want, wst = orc.prefill_quadratic(q.numpy(), k.numpy(), v.numpy(), w.numpy(), "elu1", 0.0, ost0)
    outs = []
    for r, (lo, hi) in enumerate(cuts):
        o, S, z, win, pos = seqpar.finish_rank(ops, r, q[:, :, lo:hi], k[:, :, lo:hi], v[:, :, lo:hi], w, dS_all, dz_all,
                                               tails, counts, state0)
        if o is not None:
            outs.append(o)
        np.testing.assert_allclose(S.numpy(), wst.S, rtol=1e-12, atol=1e-12)
        np.testing.assert_allclose(z.numpy(), wst.z, rtol=1e-12, atol=1e-12)
        np.testing.assert_array_equal(win.numpy(), wst.win)
        np.testing.assert_array_equal(pos.numpy(), wst.pos)
    np.testing.assert_allclose(torch.cat(outs, dim=2).numpy(), want, rtol=1e-11, atol=1e-12)


def test_every_rank_count_and_ragged_or_empty_stretches():
    for T, W, world, with_state, multiple in ((40, 3, 2, False, 8), (41, 5, 3, True, 8), (7, 4, 4, False, 8),
                                              (3, 6, 2, True, 1), (64, 1, 4, False, 16), (10, 32, 3, True, 4)):
        _run_in_process(T, W, world, with_state, multiple)


CHILD = r"""
import sys
sys.path.insert(0, %r)
import numpy as np, torch
from oracle import la_oracle as orc
from paper_2406_07368_b200 import dist as ladist, seqpar
from tests.test_seqpar_cpu import OracleOps, _case
rank, world = ladist.rank_world()
ladist.init(world, backend="gloo")
T, W = 37, 4
q, k, v, w = _case(T, W)
lo, hi = seqpar.token_shard(T, rank, world, multiple=8)
o, S, z, win, pos = seqpar.sequence_parallel_prefill(OracleOps("relu", 1e-6), seqpar.TorchDistComm(), rank,
                                                     q[:, :, lo:hi], k[:, :, lo:hi], v[:, :, lo:hi], w, W)
want, wst = orc.prefill_quadratic(q.numpy(), k.numpy(), v.numpy(), w.numpy(), "relu", 1e-6)
ok = (np.allclose(o.numpy(), want[:, :, lo:hi], rtol=1e-11, atol=1e-12) and np.allclose(S.numpy(), wst.S, rtol=1e-12)
      and np.allclose(z.numpy(), wst.z, rtol=1e-12) and np.array_equal(win.numpy(), wst.win)
      and pos.tolist() == wst.pos.tolist())
open(sys.argv[1] + f"/rank{rank}.txt", "w").write(f"{rank} {lo} {hi} {ok}")
ladist.finish(world)
"""


def test_two_gloo_ranks_reproduce_the_whole_sequence(tmp_path):
    script = tmp_path / "child.py"
    script.write_text(CHILD % ROOT)
    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "WORLD_SIZE", "LOCAL_RANK", "MASTER_PORT")}
    rc = ladist.launch_local_ranks([sys.executable, str(script), str(tmp_path)], 2, timeout=180, env=env)
    assert rc == 0
    rows = [open(tmp_path / f"rank{r}.txt").read().split() for r in range(2)]
    assert rows == [["0", "0", "24", "True"], ["1", "24", "37", "True"]]
