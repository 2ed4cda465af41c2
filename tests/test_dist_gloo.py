"""The N>1 plumbing of the benchmark on CPU: two gloo ranks, barrier, MAX of the elapsed time,
SUM of the units, disjoint worker ids."""
import os
import socket
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

CHILD = r"""
import sys
sys.path.insert(0, %r)
from paper_2312_17530_b200 import dist
rank, local_rank, world = dist.init("gloo")
assert world == 2 and rank in (0, 1)
dist.barrier()
ids = dist.worker_ids(rank, 4)
assert ids == list(range(4 * rank, 4 * rank + 4))
value, t = dist.aggregate_throughput(units_this_rank=100.0 * (rank + 1), elapsed_s_this_rank=1.0 + rank)
assert t == 2.0 and value == 150.0, (value, t)
assert dist.max_over_ranks(-1.0 - rank) == -1.0
dist.barrier()
dist.finalize()
print("rank %%d ok" %% rank)
"""


def test_two_gloo_ranks():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    procs = []
    for rank in range(2):
        env = dict(os.environ, RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE="2", MASTER_ADDR="127.0.0.1",
                   MASTER_PORT=str(port))
        procs.append(subprocess.Popen([sys.executable, "-c", CHILD % ROOT], env=env, stdout=subprocess.PIPE,
                                      stderr=subprocess.STDOUT, text=True))
    for rank, p in enumerate(procs):
        out, _ = p.communicate(timeout=120)
        assert p.returncode == 0, out
        assert "rank %d ok" % rank in out


def test_single_process_needs_no_process_group():
    from paper_2312_17530_b200 import dist

    assert dist.env_world() == (0, 0, 1) or int(os.environ.get("WORLD_SIZE", "1")) > 1
    assert dist.max_over_ranks(3.5) == 3.5 and dist.aggregate_throughput(10.0, 2.0) == (5.0, 2.0)
