"""world_size=2 on CPU (gloo): the multi-process plumbing of the benchmark.

Several GPUs only ever run independent replicas of the job, so what has to work across
processes is the barrier, the max-over-ranks of the timings, the aggregate throughput, and
the rule that only rank 0 runs and prints the reference arm."""
import json
import os
import socket
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = r"""
import json, os, sys
sys.path.insert(0, os.environ["PL_ROOT"])
from paper_2609_36954_b200 import replicas
n, rank, local = replicas.init("gloo")
replicas.barrier()
slow = replicas.max_over_ranks(10.0 + 5.0 * rank)          # rank 1 is the slow replica
agg = replicas.aggregate_throughput(1e9, slow, n)
replicas.barrier()
print(json.dumps({"rank": rank, "n": n, "max_ms": slow, "agg": agg}))
replicas.finalize()
"""


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _spawn(argv, world, extra_env=None):
    port = _free_port()
    procs = []
    for rank in range(world):
        env = dict(os.environ, MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), WORLD_SIZE=str(world),
                   RANK=str(rank), LOCAL_RANK=str(rank), PL_ROOT=ROOT, OMP_NUM_THREADS="2")
        env.update(extra_env or {})
        procs.append(subprocess.Popen(argv, env=env, stdout=subprocess.PIPE, stderr=subprocess.PIPE, text=True, cwd=ROOT))
    outs = []
    for p in procs:
        out, err = p.communicate(timeout=300)
        assert p.returncode == 0, err[-2000:]
        outs.append(out)
    return outs


def test_max_over_ranks_and_aggregate_with_two_processes():
    outs = _spawn([sys.executable, "-c", WORKER], 2)
    recs = sorted((json.loads(o.strip().splitlines()[-1]) for o in outs), key=lambda r: r["rank"])
    assert [r["rank"] for r in recs] == [0, 1]
    for r in recs:
        assert r["n"] == 2
        assert r["max_ms"] == 15.0                    # the slower replica's time, on every rank
        assert abs(r["agg"] - 2 * 1e9 / 15e-3) < 1    # both replicas' units over that time


def test_reference_arm_runs_on_rank0_only():
    outs = _spawn([sys.executable, "bench.py", "--impl", "reference", "--gpus", "2", "--steps", "2", "--warmup", "1"], 2)
    lines = [o.strip() for o in outs]
    assert lines[1] == ""                              # rank 1 exits 0 without work
    rec = json.loads(lines[0].splitlines()[-1])
    assert rec["impl"] == "reference" and rec["cpu_baseline"]["kind"] == "oracle"
    assert rec["e2e"]["h2d_bytes_per_step"] == 0 and rec["value"] > 0
    assert rec["steps"] == 2 and rec["warmup"] == 1
