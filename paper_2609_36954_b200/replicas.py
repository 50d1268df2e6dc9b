"""Process-group plumbing for multi-GPU runs.

The executor emulates its R ranks inside one GPU, so several GPUs only ever run independent
replicas of the same job: there is no data-path collective between processes.  What the
processes share is bookkeeping: a barrier around the timed region and the maximum of the
per-process times.  ``backend`` is "nccl" on GPUs and "gloo" in CPU tests.
"""
from __future__ import annotations

import os

import torch
import torch.distributed as dist


def world():
    return int(os.environ.get("WORLD_SIZE", "1")), int(os.environ.get("RANK", "0")), \
        int(os.environ.get("LOCAL_RANK", "0"))


def init(backend: str | None = None):
    """Join the process group described by the torchrun environment (no-op for one process)."""
    n, rank, local = world()
    if n == 1 or dist.is_initialized():
        return n, rank, local
    os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
    if backend is None:
        backend = "nccl" if torch.cuda.is_available() else "gloo"
    if backend == "nccl":
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    else:
        dist.init_process_group(backend)
    return n, rank, local


def barrier():
    if dist.is_initialized():
        dist.barrier()


def max_over_ranks(value: float) -> float:
    """Maximum of a per-process scalar (the job's time is its slowest replica's)."""
    if not dist.is_initialized():
        return float(value)
    dev = "cuda" if dist.get_backend() == "nccl" else "cpu"
    t = torch.tensor([float(value)], dtype=torch.float64, device=dev)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def aggregate_throughput(units_per_replica: float, ms_per_step: float, n_replicas: int) -> float:
    """Whole-job throughput: every replica moves `units_per_replica` per step, the step takes
    the slowest replica's time."""
    return n_replicas * units_per_replica / (ms_per_step * 1e-3)


def finalize():
    if dist.is_initialized():
        dist.destroy_process_group()


def launch_local(n: int, argv: list, timeout_s: float = 3600.0) -> int:
    """Start n replica processes of `argv` on this node, one per GPU index, with the environment a
    launcher would give them (RANK / LOCAL_RANK / WORLD_SIZE / MASTER_ADDR / MASTER_PORT on
    127.0.0.1).  Rank 0 inherits stdout; returns the first non-zero exit code, else 0."""
    import socket
    import subprocess
    with socket.socket() as sock:
        sock.bind(("127.0.0.1", 0))
        port = sock.getsockname()[1]
    procs = []
    for rank in range(n):
        env = dict(os.environ, MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), WORLD_SIZE=str(n), RANK=str(rank),
                   LOCAL_RANK=str(rank))
        procs.append(subprocess.Popen(argv, env=env, stdout=None if rank == 0 else subprocess.DEVNULL))
    rc = 0
    for p in procs:
        try:
            code = p.wait(timeout=timeout_s)
        except subprocess.TimeoutExpired:
            p.kill()
            code = 124
        rc = rc or code
    return rc
