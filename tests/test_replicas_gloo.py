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


def test_bench_gpus_n_starts_n_replicas_itself():
    """Without a launcher, `bench.py --gpus N` must start the N replica processes itself (here with the
    self-test that needs no GPU): rank 0 prints one line for the whole job."""
    env = {k: v for k, v in os.environ.items() if k not in ("WORLD_SIZE", "RANK", "LOCAL_RANK", "MASTER_ADDR", "MASTER_PORT")}
    out = subprocess.run([sys.executable, "bench.py", "--gpus", "2", "--replica-selftest"], env=env, cwd=ROOT,
                         capture_output=True, text=True, timeout=300)
    assert out.returncode == 0, out.stderr[-2000:]
    lines = [l for l in out.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1
    rec = json.loads(lines[0])
    assert rec == {"selftest": True, "n_gpus": 2, "max_over_ranks": 2.0}


def test_bench_refuses_a_launcher_that_disagrees_with_gpus():
    env = dict(os.environ, WORLD_SIZE="3", RANK="0", LOCAL_RANK="0", MASTER_ADDR="127.0.0.1", MASTER_PORT="29999")
    out = subprocess.run([sys.executable, "bench.py", "--gpus", "2", "--replica-selftest"], env=env, cwd=ROOT,
                         capture_output=True, text=True, timeout=120)
    assert out.returncode != 0 and "disagrees with WORLD_SIZE" in out.stderr
