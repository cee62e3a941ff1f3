"""The multi-process plumbing on CPU: two gloo ranks, max / sum over ranks, unit sharding."""
import os
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = r"""
import os, sys
sys.path.insert(0, os.environ["LA_ROOT"])
from paper_2510_08318_b200 import dist
rank, world, local = dist.init_from_env("gloo")
assert world == 2
dist.barrier()
mx = dist.max_over_ranks(10.0 + rank)          # slowest rank's time
sm = dist.sum_over_ranks(100.0 * (rank + 1))   # units processed by all ranks
lo, hi = dist.shard_range(25, rank, world)
n_units = dist.sum_over_ranks(float(hi - lo))
# one file per rank: two processes printing to one pipe can interleave their lines
with open(os.path.join(os.environ["LA_OUT"], f"rank{rank}.txt"), "w") as fh:
    fh.write(f"{rank} {mx} {sm} {lo} {hi} {n_units}\n")
dist.shutdown()
"""


def test_two_gloo_ranks_reduce_and_shard(tmp_path):
    script = tmp_path / "worker.py"
    script.write_text(WORKER)
    env = dict(os.environ, LA_ROOT=ROOT, LA_OUT=str(tmp_path))
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", "2",
           "--master-addr", "127.0.0.1", "--master-port", "29617", str(script)]
    res = subprocess.run(cmd, capture_output=True, text=True, env=env, timeout=240)
    assert res.returncode == 0, res.stderr[-2000:]
    rows = sorted((tmp_path / f"rank{r}.txt").read_text().split() for r in range(2))
    assert len(rows) == 2
    for rank, row in enumerate(rows):
        assert int(row[0]) == rank
        assert float(row[1]) == 11.0 and float(row[2]) == 300.0 and float(row[5]) == 25.0
    assert (rows[0][3], rows[0][4], rows[1][3], rows[1][4]) == ("0", "13", "13", "25")


def test_single_process_is_a_no_op():
    from paper_2510_08318_b200 import dist
    assert dist.max_over_ranks(3.5) == 3.5 and dist.sum_over_ranks(2.0) == 2.0
    dist.barrier()
    assert dist.shard_range(10, 0, 1) == (0, 10)
    assert [dist.shard_range(7, r, 3) for r in range(3)] == [(0, 3), (3, 5), (5, 7)]
