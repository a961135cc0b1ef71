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


def test_bench_starts_its_own_ranks():
    """`bench.py --gpus 2` without a launcher in the environment starts two ranks of itself; --dry-run keeps the
    run on CPU (gloo) and exercises the barrier / max-over-ranks / whole-job aggregate of the real bench."""
    import json
    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "LOCAL_RANK", "WORLD_SIZE", "MASTER_ADDR", "MASTER_PORT")}
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "2", "--dry-run", "--steps", "4",
                        "--workload", "tiny"], env=env, capture_output=True, text=True, timeout=300)
    assert r.returncode == 0, r.stdout + r.stderr
    lines = [json.loads(l) for l in r.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1                                   # rank 0 alone prints
    line = lines[0]
    assert line["n_gpus"] == 2 and line["steps"] == 4 and line["scaling"] == "weak"
    # rank r pretends a step takes (r + 1) ms: the job's time is the slowest rank's, its work the sum
    assert abs(line["ms_per_step"] - 2.0) < 1e-9 and abs(line["value"] - 8 / 8e-3) < 1e-6
    assert line["config"]["parallelism"] == "replicas x2"
