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


SPAWNED = r"""
import os, sys, time
sys.path.insert(0, %r)
from paper_2406_07368_b200 import dist as ladist
rank, world = ladist.rank_world()
out = sys.argv[1]
if len(sys.argv) > 2 and rank == int(sys.argv[2]):
    sys.exit(7)                                  # this rank fails on the host before it joins
ladist.init(world, backend="gloo")
ladist.barrier(world)
slow = ladist.max_over_ranks(3.0 + 2 * rank, world)
with open(os.path.join(out, f"rank{rank}.txt"), "w") as f:
    f.write(f"{rank} {world} {slow} {os.environ['LOCAL_RANK']} {os.environ['MASTER_ADDR']}")
ladist.finish(world)
"""


def test_the_launcher_starts_one_rank_per_gpu_and_they_agree(tmp_path):
    """What `bench.py --gpus 2` does when it is started plainly: the launcher starts the ranks itself."""
    script = tmp_path / "child.py"
    script.write_text(SPAWNED % ROOT)
    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "WORLD_SIZE", "LOCAL_RANK", "MASTER_PORT")}
    rc = ladist.launch_local_ranks([sys.executable, str(script), str(tmp_path)], 2, timeout=120, env=env)
    assert rc == 0
    rows = [open(tmp_path / f"rank{r}.txt").read().split() for r in range(2)]
    assert rows == [["0", "2", "5.0", "0", "127.0.0.1"], ["1", "2", "5.0", "1", "127.0.0.1"]]


def test_the_launcher_reports_a_rank_that_fails_and_ends_the_others(tmp_path):
    script = tmp_path / "child.py"
    script.write_text(SPAWNED % ROOT)
    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "WORLD_SIZE", "LOCAL_RANK", "MASTER_PORT")}
    rc = ladist.launch_local_ranks([sys.executable, str(script), str(tmp_path), "1"], 2, timeout=120, env=env)
    assert rc == 7
    assert not os.path.exists(tmp_path / "rank0.txt")        # rank 0 was waiting for its peer and was ended
