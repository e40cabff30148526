"""The replicated-run plumbing on CPU: two gloo ranks agree on the slowest time; shards tile the units."""
import os
import socket
import subprocess
import sys

from paper_2406_07368_b200 import dist as ladist

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

CHILD = r"""
import sys
sys.path.insert(0, %r)
from paper_2406_07368_b200 import dist as ladist
rank, world = ladist.rank_world()
ladist.init(world, backend="gloo")
ladist.barrier(world)
slow = ladist.max_over_ranks(10.0 + rank, world)
lo, hi = ladist.shard(7, rank, world)
print(f"RESULT {rank} {world} {slow} {lo} {hi}", flush=True)
ladist.finish(world)
"""


def test_shards_tile_the_units():
    for n in (1, 7, 128, 2048):
        for world in (1, 2, 3, 8):
            cuts = [ladist.shard(n, r, world) for r in range(world)]
            assert cuts[0][0] == 0 and cuts[-1][1] == n
            assert all(cuts[i][1] == cuts[i + 1][0] for i in range(world - 1))
            sizes = [b - a for a, b in cuts]
            assert max(sizes) - min(sizes) <= 1


def test_two_gloo_ranks_agree_on_the_slowest_time():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    procs = []
    for r in range(2):
        env = dict(os.environ, RANK=str(r), WORLD_SIZE="2", MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
        procs.append(subprocess.Popen([sys.executable, "-c", CHILD % ROOT], env=env, stdout=subprocess.PIPE, text=True))
    outs = [p.communicate(timeout=120)[0] for p in procs]
    assert all(p.returncode == 0 for p in procs)
    rows = sorted(line.split()[1:] for o in outs for line in o.splitlines() if line.startswith("RESULT"))
    assert rows == [["0", "2", "11.0", "0", "4"], ["1", "2", "11.0", "4", "7"]]
