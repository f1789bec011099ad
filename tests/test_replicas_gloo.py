"""Two CPU ranks over gloo exercise the multi-GPU bookkeeping of bench.py: replicas are
independent, elapsed times reduce with MAX, throughput sums the replicas' units."""
import os
import socket
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = r"""
import os, sys
sys.path.insert(0, %r)
from paper_2608_27514_b200 import replicas
rank, local_rank, n = replicas.world()
assert n == 2 and replicas.init("gloo") == 2
replicas.barrier()
mine = [1.0 + rank, 10.0 - rank]                 # rank 0: [1, 10], rank 1: [2, 9]
assert replicas.max_over_ranks(mine) == [2.0, 10.0]
rate, slowest = replicas.aggregate_throughput(256, 0.001 * (1 + rank))
assert abs(slowest - 0.002) < 1e-12 and abs(rate - 2 * 256 / 0.002) < 1e-6
replicas.barrier()
replicas.shutdown()
print("rank", rank, "ok")
""" % ROOT


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def test_two_ranks_reduce_times_with_max():
    port = str(_free_port())
    procs = []
    for rank in range(2):
        env = dict(os.environ, RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE="2",
                   MASTER_ADDR="127.0.0.1", MASTER_PORT=port)
        procs.append(subprocess.Popen([sys.executable, "-c", WORKER], env=env, stdout=subprocess.PIPE,
                                      stderr=subprocess.STDOUT, text=True))
    outs = [p.communicate(timeout=120)[0] for p in procs]
    for rank, (p, out) in enumerate(zip(procs, outs)):
        assert p.returncode == 0, out
        assert "rank %d ok" % rank in out


def test_single_process_is_identity():
    from paper_2608_27514_b200 import replicas
    for k in ("RANK", "LOCAL_RANK", "WORLD_SIZE"):
        os.environ.pop(k, None)
    assert replicas.world() == (0, 0, 1)
    assert replicas.max_over_ranks([3.5, 1.0]) == [3.5, 1.0]
    assert replicas.aggregate_throughput(100, 0.5) == (200.0, 0.5)
