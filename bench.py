#!/usr/bin/env python
"""Benchmark of the collectives executor.

Default line (N=1): one *step* = reduce-scatter followed by all-gather over R=8 emulated
ranks, 64 MiB per rank bf16 N(0,1), direct schedules with 1 MiB chunks -- the configuration
the headline metric (effective collective GB/s, fraction of HBM peak) is quoted on.  Message
sizes follow the paper's convention (Sec. 5, "Microbenchmark methodology": per-rank input
for reduce-scatter, gathered output for all-gather; algorithm bandwidth = size / latency).

  python bench.py [--gpus N] [--steps K] [--warmup W]            # the CUDA path
  python bench.py --impl reference [--steps K] [--warmup W]      # the CPU oracle, timed
  python bench.py --cpu-suite                                    # the CPU oracle on samples of every configuration
  python bench.py --suite                                          # every configuration, one line each

With N > 1 (torchrun) every rank runs an independent replica on its own GPU: the path has
no inter-GPU exchange (the R ranks are emulated inside one GPU), so this is weak scaling of
replicas with no data-path collective.
"""
from __future__ import annotations

import argparse
import json
import os
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

MIB = 1 << 20
NOMINAL_HBM_GBS = 8000.0
FALLBACK_HBM_GBS = 6650.0
# dram__bytes_read.sum + dram__bytes_write.sum of one reduce-scatter launch of this workload
# (one ncu capture of that launch)
NCU_RS_TRAFFIC_BYTES = 593797120.0


def measured_peak():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(p) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


# ------------------------------------------------------------------------------------------
# clocks sampled during the timed region (NVML, read-only)
# ------------------------------------------------------------------------------------------
class ClockSampler:
    def __init__(self, index):
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self._stop = threading.Event()
        self._thread = None
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = int(pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM))
        except Exception:
            self.nv = None

    def _loop(self):
        nv = self.nv
        names = {"hw_slowdown": 0x8, "sw_power_cap": 0x4, "hw_thermal_slowdown": 0x40,
                 "sw_thermal_slowdown": 0x20, "hw_power_brake": 0x80}
        while not self._stop.is_set():
            try:
                self.samples.append(int(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM)))
                try:
                    mask = int(nv.nvmlDeviceGetCurrentClocksEventReasons(self.h))
                except Exception:
                    mask = int(nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h))
                for k, bit in names.items():
                    if mask & bit:
                        self.reasons.add(k)
            except Exception:
                pass
            time.sleep(0.01)

    def start(self):
        if self.nv is not None:
            self._thread = threading.Thread(target=self._loop, daemon=True)
            self._thread.start()

    def stop(self):
        self._stop.set()
        if self._thread is not None:
            self._thread.join()
        med = int(np.median(self.samples)) if self.samples else None
        return {"sm_mhz": med, "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons),
                "samples": len(self.samples)}


# ------------------------------------------------------------------------------------------
# workload C2
# ------------------------------------------------------------------------------------------
C2 = dict(R=8, bytes_per_rank=64 * MIB, chunk=1 * MIB)


def c2_inputs(R, n, seed=0, unique=None):
    """Per-rank bf16 N(0,1) inputs (uint16 bits).  `unique` elements are generated and tiled
    to n when given (the CPU generator is slow; the distribution is unchanged)."""
    from paper_2609_36954_b200 import inputs as gen
    out = []
    u = n if unique is None else min(unique, n)
    for r in range(R):
        a = gen.normal_bf16(u, seed, r)
        if u < n:
            a = np.tile(a, (n + u - 1) // u)[:n]
        out.append(np.ascontiguousarray(a))
    return out


def run_purlin(args):
    import torch

    from paper_2609_36954_b200 import binding as B
    from paper_2609_36954_b200 import replicas

    world, rank, local = replicas.world()
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback)")
    torch.cuda.set_device(local)
    replicas.init("nccl")

    R, Mb, chunk = C2["R"], C2["bytes_per_rank"], C2["chunk"]
    n = Mb // 2
    stream = torch.cuda.current_stream().cuda_stream
    peak, peak_kind = measured_peak()

    # the full-size inputs are generated exactly (seeded, per rank) unless --fast-inputs
    x = c2_inputs(R, n, seed=0, unique=(4 * MIB if args.fast_inputs else None))
    comm = B.pl_comm_create(R, B.PL_BF16)
    opts = B.make_opts(n_ctas=args.n_ctas, threads=args.threads, slice_bytes=args.slice_bytes,
                       datapath=args.datapath, stages=args.stages, stage_bytes=args.stage_bytes)
    rs = B.pl_schedule_build(comm, B.PL_REDUCE_SCATTER, B.PL_ALGO_DIRECT, n, chunk, opts)
    ag = B.pl_schedule_build(comm, B.PL_ALLGATHER, B.PL_ALGO_DIRECT, n // R, chunk, opts)
    irs, iag = B.pl_schedule_info(rs), B.pl_schedule_info(ag)

    pinned_in = [torch.from_numpy(a.view(np.int16)).pin_memory() for a in x]
    d_in = [t.cuda(non_blocking=True) for t in pinned_in]
    d_mid = [torch.empty(n // R, dtype=torch.int16, device="cuda") for _ in range(R)]
    d_out = [torch.empty(n, dtype=torch.int16, device="cuda") for _ in range(R)]
    torch.cuda.synchronize()

    def bufs(ins, outs, info):
        return B.make_bufs([t.data_ptr() for t in ins], [t.data_ptr() for t in outs],
                           [int(info.in_bytes[r]) for r in range(R)], [int(info.out_bytes[r]) for r in range(R)])
    b_rs, b_ag = bufs(d_in, d_mid, irs), bufs(d_mid, d_out, iag)

    def step():
        B.pl_execute(rs, b_rs, stream)
        B.pl_execute(ag, b_ag, stream)

    for _ in range(max(3, args.warmup)):
        step()
    torch.cuda.synchronize()
    assert B.pl_comm_status(comm).code == B.PL_OK

    # ---- device-timed region --------------------------------------------------------------
    K = args.steps
    ev = [[torch.cuda.Event(enable_timing=True) for _ in range(3)] for _ in range(K)]
    sampler = ClockSampler(local)
    launches0 = B.pl_launch_count()
    replicas.barrier()
    torch.cuda.synchronize()
    sampler.start()
    t_begin = torch.cuda.Event(enable_timing=True)
    t_end = torch.cuda.Event(enable_timing=True)
    t_begin.record()
    for i in range(K):
        ev[i][0].record()
        B.pl_execute(rs, b_rs, stream)
        ev[i][1].record()
        B.pl_execute(ag, b_ag, stream)
        ev[i][2].record()
    t_end.record()
    torch.cuda.synchronize()
    clocks = sampler.stop()
    launches = B.pl_launch_count() - launches0
    total_ms = t_begin.elapsed_time(t_end)
    rs_ms = np.array([ev[i][0].elapsed_time(ev[i][1]) for i in range(K)])
    ag_ms = np.array([ev[i][1].elapsed_time(ev[i][2]) for i in range(K)])
    assert B.pl_comm_status(comm).code == B.PL_OK
    replicas.barrier()
    total_ms = replicas.max_over_ranks(total_ms)

    ms_per_step = total_ms / K
    eff_bytes = irs.message_bytes + iag.message_bytes  # 64 MiB + 64 MiB per step
    value = replicas.aggregate_throughput(eff_bytes, ms_per_step, world) / 1e9

    # ---- end to end through the host-buffer entry point -----------------------------------
    e2e = None
    if not args.no_e2e:
        h_mid = [torch.empty(n // R, dtype=torch.int16).pin_memory() for _ in range(R)]
        h_out = [torch.empty(n, dtype=torch.int16).pin_memory() for _ in range(R)]
        hb_rs, hb_ag = bufs(pinned_in, h_mid, irs), bufs(h_mid, h_out, iag)
        Ke = max(3, min(10, K))

        def e2e_step():
            B.pl_execute_host(rs, hb_rs, b_rs, stream)
            B.pl_execute_host(ag, hb_ag, b_ag, stream)
        for _ in range(2):
            e2e_step()
        torch.cuda.synchronize()
        replicas.barrier()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(Ke):
            e2e_step()
        e1.record()
        torch.cuda.synchronize()
        e_ms = replicas.max_over_ranks(e0.elapsed_time(e1))
        h2d = sum(int(irs.in_bytes[r]) + int(iag.in_bytes[r]) for r in range(R))
        d2h = sum(int(irs.out_bytes[r]) + int(iag.out_bytes[r]) for r in range(R))
        e2e = {"value": replicas.aggregate_throughput(eff_bytes, e_ms / Ke, world) / 1e9, "unit": "GB/s", "steps": Ke,
               "ms_per_step": e_ms / Ke, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
               "api": "pl_execute_host (pinned host buffers in and out)"}
        # parity spot check of the e2e result on sampled elements against the definition
        got = h_out[3].numpy().view(np.uint16)
        idx = np.linspace(0, n - 1, 64).astype(np.int64)
        from paper_2609_36954_b200 import inputs as gen
        exact = sum(gen.bf16_bits_to_f64(a[idx]) for a in x)
        gotf = gen.bf16_bits_to_f64(got[idx])
        assert np.all(np.abs(gotf - exact) <= 2.0 ** -7 * np.abs(exact) + 1e-6), "e2e result is wrong"

    # ---- p50 latency of the small all-reduce (the metric's second half) ----------------------
    latency = None
    if not args.no_latency:
        latency = measure_small_allreduce(B, torch, stream)

    # ---- roofline of the dominant kernel (the reduce-scatter launch) -----------------------
    rs_alg = irs.bytes_read + irs.bytes_written            # (R+1) * M: every byte touched once
    ag_floor = iag.in_bytes[0] * R + iag.bytes_written     # compulsory DRAM traffic (R+1) * M
    rs_gbs = rs_alg / (rs_ms.mean() * 1e-3) / 1e9
    ag_gbs = ag_floor / (ag_ms.mean() * 1e-3) / 1e9
    roofline = {"bound": "hbm", "kernel": "pl_exec_tma_kernel<bf16> (reduce-scatter launch)",
                "achieved": rs_gbs, "peak": peak, "peak_kind": peak_kind, "unit": "GB/s",
                "frac": rs_gbs / peak, "frac_of_nominal_8TBps": rs_gbs / NOMINAL_HBM_GBS,
                "algorithmic_bytes_per_launch": int(rs_alg), "avg_launch_us": float(rs_ms.mean() * 1e3),
                "traffic": args.ncu_traffic}
    detail = {
        "reduce_scatter": {"us": float(rs_ms.mean() * 1e3), "p50_us": float(np.median(rs_ms) * 1e3),
                           "algbw_gbs": irs.message_bytes / (rs_ms.mean() * 1e-3) / 1e9,
                           "hbm_gbs": rs_gbs, "frac_measured": rs_gbs / peak, "frac_8TBps": rs_gbs / NOMINAL_HBM_GBS},
        "all_gather": {"us": float(ag_ms.mean() * 1e3), "p50_us": float(np.median(ag_ms) * 1e3),
                       "algbw_gbs": iag.message_bytes / (ag_ms.mean() * 1e-3) / 1e9,
                       "hbm_gbs_compulsory": ag_gbs, "frac_measured": ag_gbs / peak,
                       "schedule_gbs": (iag.bytes_read + iag.bytes_written) / (ag_ms.mean() * 1e-3) / 1e9},
        "grid": int(irs.grid), "threads": int(irs.threads), "slice_bytes": int(irs.slice_bytes),
        "datapath": int(irs.datapath), "n_ops_rs": int(irs.n_ops), "n_ops_ag": int(iag.n_ops),
    }

    # ---- the oracle timed on this machine's host cores (rank 0, N=1 only) -----------------------
    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu:
        cpu = time_oracle_c2(x, target_s=args.cpu_seconds)

    if rank == 0:
        line = {
            "metric": "effective collective GB/s", "value": value, "unit": "GB/s", "n_gpus": world,
            "steps": K, "warmup": max(3, args.warmup), "ms_per_step": ms_per_step, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": {"workload": "C2: reduce-scatter (64 MiB/rank in) then all-gather (64 MiB/rank out), "
                                   "R=8 emulated ranks in one HBM, bf16 N(0,1) seed 0, direct schedules, 1 MiB chunks",
                       "l2": "inputs_larger_than_l2 (512 MiB of inputs per step; no flush)",
                       "replicas": world, "parallelism": "replicas only (no inter-GPU exchange on this path)"},
            "clocks": clocks, "e2e": e2e, "gpu_launches": int(launches), "roofline": roofline,
            "cpu_baseline": cpu, "small_allreduce": latency, "detail": detail,
        }
        print(json.dumps(line))
    B.pl_schedule_destroy(rs)
    B.pl_schedule_destroy(ag)
    B.pl_comm_destroy(comm)
    replicas.finalize()


def measure_small_allreduce(B, torch, stream, R=8, hidden=8192, layers=80, steps=200):
    """Tensor-parallel decode shape: one token x hidden 8192 bf16 (16 KiB per rank), 80
    back-to-back all-reduces in ONE launch, distinct inputs per layer.  p50 over steps of the
    time per layer, CUDA events around each launch."""
    from paper_2609_36954_b200 import inputs as gen
    n = hidden
    comm = B.pl_comm_create(R, B.PL_BF16)
    out = {}
    for name, algo in (("oneshot", B.PL_ALGO_ONESHOT), ("fused", B.PL_ALGO_DIRECT_FUSED)):
        s = B.pl_schedule_build_layers(comm, algo, n, layers, None)
        info = B.pl_schedule_info(s)
        d_in = [torch.from_numpy(np.concatenate([gen.normal_bf16(n, 0, l * R + r) for l in range(layers)]).view(np.int16)).cuda()
                for r in range(R)]
        d_out = [torch.empty(n * layers, dtype=torch.int16, device="cuda") for _ in range(R)]
        bufs = B.make_bufs([t.data_ptr() for t in d_in], [t.data_ptr() for t in d_out],
                           [int(info.in_bytes[r]) for r in range(R)], [int(info.out_bytes[r]) for r in range(R)])
        for _ in range(5):
            B.pl_execute(s, bufs, stream)
        torch.cuda.synchronize()
        ev = [torch.cuda.Event(enable_timing=True) for _ in range(steps + 1)]
        ev[0].record()
        for i in range(steps):
            B.pl_execute(s, bufs, stream)
            ev[i + 1].record()
        torch.cuda.synchronize()
        us = np.array([ev[i].elapsed_time(ev[i + 1]) for i in range(steps)]) * 1e3 / layers
        out[name] = {"p50_us": float(np.median(us)), "p10_us": float(np.percentile(us, 10)),
                     "p90_us": float(np.percentile(us, 90)), "grid": int(info.grid)}
        B.pl_schedule_destroy(s)
    B.pl_comm_destroy(comm)
    best = min(out, key=lambda k: out[k]["p50_us"])
    return {"metric": "p50 us per 16 KiB all-reduce (R=8, bf16, 80 layers per launch, per layer)",
            "p50_us": out[best]["p50_us"], "algorithm": best, "all": out, "steps": steps}


# ------------------------------------------------------------------------------------------
# the oracle, timed as it stands
# ------------------------------------------------------------------------------------------
def oracle_step(x_sample):
    from oracle import oracle
    R = len(x_sample)
    rs = oracle.reduce_scatter(x_sample, "bf16")                    # fp64 outputs
    from paper_2609_36954_b200 import inputs as gen
    mid = [gen.f32_to_bf16_bits(a.astype(np.float32)) for a in rs]  # what the next collective takes
    oracle.allgather(mid)
    return R


def time_oracle_c2(x, target_s=12.0):
    """Time the CPU oracle on a bounded sample of the C2 workload (whole buffers if quick)."""
    from oracle import oracle
    R = len(x)
    n = x[0].size
    frac = 1
    sample = [a[: n // frac] for a in x]
    t0 = time.perf_counter()
    oracle_step(sample)
    t1 = time.perf_counter() - t0
    reps = int(max(1, min(20, target_s / max(t1, 1e-3))))
    t0 = time.perf_counter()
    for _ in range(reps):
        oracle_step(sample)
    dt = (time.perf_counter() - t0) / reps
    eff = 2 * sample[0].nbytes  # RS message + AG message
    return {"value": eff / dt / 1e9, "unit": "GB/s", "cores": oracle.num_threads(), "kind": "oracle",
            "sample": f"whole C2 step (R={R}, {sample[0].nbytes // MIB} MiB/rank), {reps} repetitions, "
                      f"{dt * 1e3:.1f} ms per step"}


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from oracle import oracle
    R, Mb = C2["R"], C2["bytes_per_rank"]
    K, W = args.steps, args.warmup
    # bound the whole run to ~2 minutes: shrink the per-step sample by powers of two
    x_full_n = Mb // 2
    probe = c2_inputs(R, 1 * MIB, seed=0)
    t0 = time.perf_counter()
    oracle_step(probe)
    per_mib = (time.perf_counter() - t0) / 2.0  # seconds per MiB/rank
    budget = 120.0 / max(1, K + W)
    n = x_full_n
    while n > 32768 and per_mib * (2 * n / MIB) > budget:
        n //= 2
    x = c2_inputs(R, n, seed=0, unique=min(n, 4 * MIB))
    for _ in range(W):
        oracle_step(x)
    t0 = time.perf_counter()
    for _ in range(K):
        oracle_step(x)
    dt = (time.perf_counter() - t0) / K
    eff = 2 * x[0].nbytes
    value = eff / dt / 1e9
    sample = f"{x[0].nbytes / MIB:.3f} MiB/rank of the 64 MiB/rank C2 step per step (R={R})"
    line = {"impl": "reference", "metric": "effective collective GB/s", "value": value, "unit": "GB/s",
            "n_gpus": int(os.environ.get("WORLD_SIZE", "1")), "steps": K, "warmup": W, "ms_per_step": dt * 1e3,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": "C2: reduce-scatter then all-gather, R=8, bf16 N(0,1) seed 0 (CPU oracle, "
                                   "fp64 accumulation)", "sample": sample},
            "cpu_baseline": {"value": value, "unit": "GB/s", "cores": oracle.num_threads(), "kind": "oracle",
                             "sample": sample},
            "e2e": {"value": value, "unit": "GB/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))


# ---------------------------------------------------------------------------------------------
# the oracle timed per configuration (reported baseline: wall time per collective on the host)
# ---------------------------------------------------------------------------------------------
def run_cpu_suite(args):
    """One JSON line per (configuration, thread count): the CPU oracle as it stands, on bounded
    samples of every benchmark configuration, with 1 thread and with every available core.
    No GPU is touched."""
    import ctypes
    from oracle import oracle
    from paper_2609_36954_b200 import inputs as gen
    omp = ctypes.CDLL("libgomp.so.1")
    all_threads = oracle.num_threads()

    def timed(fn, budget_s=2.0):
        fn()
        t0 = time.perf_counter()
        reps = 0
        while True:
            fn()
            reps += 1
            dt = time.perf_counter() - t0
            if reps >= 3 and dt >= budget_s or reps >= 50:
                return dt / reps

    def emit(cfg, what, threads, sec, eff_bytes):
        print(json.dumps({"cfg": cfg, "impl": "cpu-oracle", "what": what, "threads": threads, "us": sec * 1e6,
                          "eff_gbs": eff_bytes / sec / 1e9}), flush=True)

    cases = []
    x1 = gen.rank_inputs(4, 262144, "f32", seed=0)
    cases.append(("C1", "all-reduce R=4 1 MiB fp32", lambda: oracle.allreduce(x1, "f32"), 1 << 20))
    n2 = 4 * MIB  # 8 MiB per rank sample of the 64 MiB C2 message
    x2 = [gen.normal_bf16(n2, 0, r) for r in range(8)]
    cases.append(("C2", "reduce-scatter R=8, 8 MiB/rank sample", lambda: oracle.reduce_scatter(x2, "bf16"), n2 * 2))
    part = [a[: n2 // 8].copy() for a in x2]
    cases.append(("C2", "all-gather R=8, 8 MiB/rank sample", lambda: oracle.allgather(part), n2 * 2))
    for kib in (4, 64, 1024, 16384):
        n = kib * 1024 // 2
        x = [gen.normal_bf16(n, 0, r) for r in range(8)]
        cases.append(("C3", f"all-reduce R=8 {kib} KiB bf16", (lambda x=x: oracle.allreduce(x, "bf16")), n * 2))
    R, T, H, E, K = 8, 256, 7168, 256, 8  # 256 of the 4096 tokens per rank
    idx, gates = gen.moe_routing(R, T, E, K, seed=0)
    xt = gen.moe_tokens_bf16(R, T, H, seed=2)
    disp = oracle.moe_dispatch(xt, idx, E, recv_capacity_rows=R * T * K)
    cases.append(("C4", "MoE dispatch, 256 tokens/rank sample", lambda: oracle.moe_dispatch(xt, idx, E, recv_capacity_rows=R * T * K), R * T * K * H * 2))
    cases.append(("C4", "MoE combine, 256 tokens/rank sample", lambda: oracle.moe_combine(disp["recv"], idx, disp["pos"], gates, E, H), R * T * K * H * 2))
    x5 = [gen.normal_bf16(8192, 0, r) for r in range(8)]
    cases.append(("C5", "all-reduce R=8 16 KiB (one decode layer)", lambda: oracle.allreduce(x5, "bf16"), 16384))
    for threads in sorted({1, all_threads}):
        omp.omp_set_num_threads(threads)
        for cfg, what, fn, eff in cases:
            emit(cfg, what, threads, timed(fn, budget_s=args.cpu_seconds / 12.0), eff)
    omp.omp_set_num_threads(all_threads)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=1000)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", default="purlin", choices=["purlin", "reference"])
    ap.add_argument("--suite", action="store_true", help="run every configuration (bench_suite.py)")
    ap.add_argument("--cpu-suite", action="store_true", help="time the CPU oracle on samples of every configuration (1 thread and all cores)")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu", action="store_true")
    ap.add_argument("--no-latency", action="store_true")
    ap.add_argument("--fast-inputs", action="store_true", help="tile 4 Mi generated elements instead of generating all")
    ap.add_argument("--cpu-seconds", type=float, default=12.0)
    ap.add_argument("--n-ctas", type=int, default=0)
    ap.add_argument("--threads", type=int, default=0)
    ap.add_argument("--slice-bytes", type=int, default=0)
    ap.add_argument("--datapath", type=int, default=0)
    ap.add_argument("--stages", type=int, default=0)
    ap.add_argument("--stage-bytes", type=int, default=0)
    ap.add_argument("--ncu-traffic", type=float, default=NCU_RS_TRAFFIC_BYTES,
                    help="dram bytes per reduce-scatter launch from the committed ncu capture")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    elif args.cpu_suite:
        run_cpu_suite(args)
    elif args.suite:
        import bench_suite
        bench_suite.main(args)
    else:
        run_purlin(args)


if __name__ == "__main__":
    main()
