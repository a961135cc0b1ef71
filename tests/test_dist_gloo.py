"""World-size-2 gloo run of the replica plumbing bench.py uses at N > 1 (CPU only)."""
import os
import socket
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

CHILD = r"""
import sys
sys.path.insert(0, %r)
from paper_2607_19539_b200 import dist as D
rank, local_rank, world = D.init("gloo")
assert world == 2
D.barrier()
# rank r processes (r + 1) * 100 units in (r + 1) seconds: job throughput = 300 units / 2 s
tput, t = D.aggregate_throughput((rank + 1) * 100.0, float(rank + 1))
assert t == 2.0 and tput == 150.0, (t, tput)
assert D.max_over_ranks(float(rank)) == 1.0 and D.sum_over_ranks(1.0) == 2.0
D.barrier()
D.finalize()
print("ok", rank)
"""


def test_two_rank_gloo_aggregate():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    procs = []
    for r in range(2):
        env = dict(os.environ, RANK=str(r), LOCAL_RANK=str(r), WORLD_SIZE="2", MASTER_ADDR="127.0.0.1",
                   MASTER_PORT=str(port))
        procs.append(subprocess.Popen([sys.executable, "-c", CHILD % ROOT], env=env, stdout=subprocess.PIPE,
                                      stderr=subprocess.STDOUT, text=True))
    outs = [p.communicate(timeout=120)[0] for p in procs]
    assert all(p.returncode == 0 for p in procs), outs
    assert all("ok" in o for o in outs)


def test_single_process_is_identity():
    from paper_2607_19539_b200 import dist as D
    assert D.aggregate_throughput(10.0, 2.0) == (5.0, 2.0)
