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
# (one ncu capture of that launch, caches flushed before it: 537.7 MB read, 18.1 MB written; three
# quarters of the 64 MiB of results are still in L2 when the kernel ends)
NCU_RS_TRAFFIC_BYTES = 555785728.0
# the same sum for a reduce-scatter launch inside the step (one pass, caches left as the
# all-gather before it left them): 537.1 MB read, 76.9 MB written
NCU_RS_TRAFFIC_IN_SITU_BYTES = 614000000.0


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
    # set-up: which grid this GPU's memory system serves the all-gather's 1 read : 8 writes stream best with
    tuned_grid = 0 if (args.no_tune or args.ag_grid) else B.pl_comm_tune(comm, stream)   # later builds on comm use what it measured
    # Both launches read their inputs for the last time (the reduce-scatter consumes the
    # contributions, the all-gather the reduced partition): PL_OPT_INPUTS_LAST_USE says so.
    step_flags = 0 if args.plain_options else B.PL_OPT_INPUTS_LAST_USE
    opts = B.make_opts(n_ctas=args.n_ctas, threads=args.threads, slice_bytes=args.slice_bytes,
                       datapath=args.datapath, stages=args.stages, stage_bytes=args.stage_bytes, flags=step_flags)
    # The reduce-scatter is also launched overlapped: its CTAs are set up (barriers, first
    # descriptor) while the all-gather in front of it drains, 2 us per step.  The all-gather is
    # not: CTAs of an overlapped launch take the SMs in the order in which they become free, and a
    # grid smaller than the SM count then ends up on other SMs than the ones it was tuned for (+7 us).
    opts_rs = opts if args.plain_options else B.make_opts(
        n_ctas=args.n_ctas, threads=args.threads, slice_bytes=args.slice_bytes, datapath=args.datapath, stages=args.stages,
        stage_bytes=args.stage_bytes, flags=step_flags | B.PL_OPT_OVERLAP_LAUNCH)
    rs = B.pl_schedule_build(comm, B.PL_REDUCE_SCATTER, B.PL_ALGO_DIRECT, n, chunk, opts_rs)
    if args.ag_grid:    # profiling runs: the all-gather's grid given instead of measured (no tuning launches)
        first, count = (int(v) for v in args.ag_idle.split(":")) if args.ag_idle else (0, 0)
        opts_ag = B.make_opts(n_ctas=args.ag_grid, threads=args.threads, slice_bytes=args.slice_bytes, datapath=args.datapath,
                              stages=args.stages, stage_bytes=args.stage_bytes, flags=step_flags, idle_sm_first=first, idle_sm_count=count)
    else:
        opts_ag = opts
    ag = B.pl_schedule_build(comm, B.PL_ALLGATHER, B.PL_ALGO_DIRECT, n // R, chunk, opts_ag)
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
    # A block is exactly K steps bracketed by a barrier and a device synchronisation on both
    # sides.  The block is repeated until the timed region lasts at least half a second, so that
    # the clock record holds more than one sample whatever K is; the median block is reported.
    K = args.steps
    sampler = ClockSampler(local)
    launches0 = B.pl_launch_count()

    def one_block(inner_events):
        """K steps between a barrier + device synchronisation on both sides.  Without inner
        events the block is what a caller runs (launch after launch) and gives the step time;
        with an event between all launches it gives each launch's duration, at the price of
        about 2.5 us per launch that the event itself puts between two kernels."""
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        ev = [[torch.cuda.Event(enable_timing=True) for _ in range(3)] for _ in range(K)] if inner_events else None
        replicas.barrier()
        torch.cuda.synchronize()
        e0.record()
        for i in range(K):
            if ev:
                ev[i][0].record()
            B.pl_execute(rs, b_rs, stream)
            if ev:
                ev[i][1].record()
            B.pl_execute(ag, b_ag, stream)
            if ev:
                ev[i][2].record()
        e1.record()
        torch.cuda.synchronize()
        replicas.barrier()
        if not ev:
            return e0.elapsed_time(e1), [], []
        return (e0.elapsed_time(e1),
                [ev[i][0].elapsed_time(ev[i][1]) for i in range(K)], [ev[i][1].elapsed_time(ev[i][2]) for i in range(K)])

    sampler.start()
    block_ms, block_ms_events, rs_all, ag_all = [], [], [], []
    spent = 0.0
    while True:
        # blocks alternate: plain (the step time) and with per-launch events (the launch durations)
        inner = len(block_ms) > len(block_ms_events)
        ms, r_ms, a_ms = one_block(inner)
        ms = replicas.max_over_ranks(ms)               # the job's block time is its slowest replica's
        (block_ms_events if inner else block_ms).append(ms)
        rs_all += r_ms
        ag_all += a_ms
        spent += ms
        if (spent >= args.min_timed_ms and len(block_ms_events) >= 1) or len(block_ms) >= 1000:
            break
    clocks = sampler.stop()
    n_blocks = len(block_ms)
    launches = (B.pl_launch_count() - launches0) // (n_blocks + len(block_ms_events))      # kernels launched per timed block of K steps
    total_ms = float(np.median(block_ms))
    rs_ms, ag_ms = np.array(rs_all), np.array(ag_all)
    assert B.pl_comm_status(comm).code == B.PL_OK

    ms_per_step = total_ms / K
    eff_bytes = irs.message_bytes + iag.message_bytes  # 64 MiB + 64 MiB per step
    value = replicas.aggregate_throughput(eff_bytes, ms_per_step, world) / 1e9

    # ---- end to end through the host-buffer entry point -----------------------------------
    e2e = None
    if not args.no_e2e:
        h_mid = [torch.empty(n // R, dtype=torch.int16).pin_memory() for _ in range(R)]
        h_out = [torch.empty(n, dtype=torch.int16).pin_memory() for _ in range(R)]
        hb_rs, hb_ag = bufs(pinned_in, h_mid, irs), bufs(h_mid, h_out, iag)
        Ke = max(3, min(20, K))

        # the pipelined host entry point: the download of one call overlaps the upload of the next
        def e2e_step():
            B.pl_execute_host_async(rs, hb_rs, b_rs, stream)
            B.pl_execute_host_async(ag, hb_ag, b_ag, stream)
        for _ in range(2):
            e2e_step()
        B.pl_comm_host_sync(comm)
        torch.cuda.synchronize()
        replicas.barrier()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        copied0 = B.pl_comm_host_stats(comm)
        e0.record()
        for _ in range(Ke):
            e2e_step()
        B.pl_comm_host_fence(comm, stream)     # the timed region ends when the last download has landed
        e1.record()
        torch.cuda.synchronize()
        e_ms = replicas.max_over_ranks(e0.elapsed_time(e1))
        # bytes actually copied per step, from the library's own count: the all-gather's input is
        # the reduce-scatter's result, handed over through a host buffer while its download is in
        # flight, so it is not uploaded again (it is already in the device buffer it came from)
        copied1 = B.pl_comm_host_stats(comm)
        h2d = (copied1[0] - copied0[0]) // Ke
        d2h = (copied1[1] - copied0[1]) // Ke
        e2e = {"value": replicas.aggregate_throughput(eff_bytes, e_ms / Ke, world) / 1e9, "unit": "GB/s", "steps": Ke,
               "ms_per_step": e_ms / Ke, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
               "api": "pl_execute_host_async (pinned host buffers in and out; uploads, schedule and downloads of "
                      "consecutive calls on three streams; an input that the previous call's download is still "
                      "writing from the same device buffer is not uploaded again)"}
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
    ag_floor = iag.hbm_bytes                               # compulsory DRAM traffic (R+1) * M
    rs_gbs = rs_alg / (rs_ms.mean() * 1e-3) / 1e9
    ag_gbs = ag_floor / (ag_ms.mean() * 1e-3) / 1e9
    roofline = {"bound": "hbm", "kernel": "pl_exec_tma_kernel<bf16> (reduce-scatter launch)",
                "achieved": rs_gbs, "peak": peak, "peak_kind": peak_kind, "unit": "GB/s",
                "frac": rs_gbs / peak, "frac_of_nominal_8TBps": rs_gbs / NOMINAL_HBM_GBS,
                "algorithmic_bytes_per_launch": int(rs_alg), "avg_launch_us": float(rs_ms.mean() * 1e3),
                "traffic": args.ncu_traffic, "traffic_in_situ": NCU_RS_TRAFFIC_IN_SITU_BYTES,
                "dram_gbs_in_situ": NCU_RS_TRAFFIC_IN_SITU_BYTES / (rs_ms.mean() * 1e-3) / 1e9}
    detail = {
        "reduce_scatter": {"us": float(rs_ms.mean() * 1e3), "p50_us": float(np.median(rs_ms) * 1e3),
                           "algbw_gbs": irs.message_bytes / (rs_ms.mean() * 1e-3) / 1e9,
                           "hbm_gbs": rs_gbs, "frac_measured": rs_gbs / peak, "frac_8TBps": rs_gbs / NOMINAL_HBM_GBS},
        "all_gather": {"us": float(ag_ms.mean() * 1e3), "p50_us": float(np.median(ag_ms) * 1e3),
                       "algbw_gbs": iag.message_bytes / (ag_ms.mean() * 1e-3) / 1e9,
                       "hbm_gbs_compulsory": ag_gbs, "frac_measured": ag_gbs / peak,
                       "schedule_gbs": (iag.bytes_read + iag.bytes_written) / (ag_ms.mean() * 1e-3) / 1e9},
        "grid": int(irs.grid), "grid_all_gather": int(iag.grid), "grid_all_gather_tuned": int(tuned_grid),
        "idle_sms_all_gather": {"first": int(iag.idle_sm_first), "count": int(iag.idle_sm_count)}, "threads": int(irs.threads), "slice_bytes": int(irs.slice_bytes),
        "datapath": int(irs.datapath), "n_ops_rs": int(irs.n_ops), "n_ops_ag": int(iag.n_ops),
    }

    detail["timed_region"] = {"blocks": n_blocks, "steps_per_block": K, "block_ms_median": total_ms,
                              "block_ms_min": float(min(block_ms)), "block_ms_max": float(max(block_ms)),
                              "blocks_with_an_event_between_launches": len(block_ms_events),
                              "their_block_ms_median": float(np.median(block_ms_events)),
                              "note": "blocks alternate: plain ones give ms_per_step and value, the ones with an event "
                                      "between all launches give the per-launch durations of roofline and detail"}

    # ---- the same step with overlapped launches (no events between the two executes) ---------
    if not args.no_detail:
        detail["step_both_launches_overlapped"] = measure_step_variant(B, torch, comm, n, chunk, R, b_rs, b_ag, stream, ms_per_step,
                                                                       step_flags | B.PL_OPT_OVERLAP_LAUNCH)
        detail["step_without_last_use_hint"] = measure_step_variant(B, torch, comm, n, chunk, R, b_rs, b_ag, stream, ms_per_step, 0)

    # free the headline buffers before the other configurations allocate theirs
    del d_in, d_mid, d_out, b_rs, b_ag, pinned_in
    torch.cuda.empty_cache()

    # ---- every other configuration, measured in this same process -----------------------------
    if rank == 0 and world == 1 and not args.no_detail:
        detail["configs"] = measure_all_configs(peak)

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
                       "options": "default" if args.plain_options else "PL_OPT_INPUTS_LAST_USE on both schedules (inputs loaded evict-first), "
                                  "PL_OPT_OVERLAP_LAUNCH on the reduce-scatter; all-gather grid from pl_comm_tune",
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


def measure_step_variant(B, torch, comm, n, chunk, R, b_rs, b_ag, stream, plain_ms, flags):
    """The C2 step built with other schedule options and timed without events between the two
    launches.  PL_OPT_OVERLAP_LAUNCH (the CTAs of a launch are set up while the one in front of it
    drains) is made for the latency path; on these HBM-bound launches it does not pay (the CTAs of
    a launch then take the SMs in the order in which they become free).  flags = 0 is the step
    without PL_OPT_INPUTS_LAST_USE."""
    opts = B.make_opts(flags=flags)
    rs = B.pl_schedule_build(comm, B.PL_REDUCE_SCATTER, B.PL_ALGO_DIRECT, n, chunk, opts)
    ag = B.pl_schedule_build(comm, B.PL_ALLGATHER, B.PL_ALGO_DIRECT, n // R, chunk, opts)
    for _ in range(5):
        B.pl_execute(rs, b_rs, stream)
        B.pl_execute(ag, b_ag, stream)
    torch.cuda.synchronize()
    reps = 300
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(reps):
        B.pl_execute(rs, b_rs, stream)
        B.pl_execute(ag, b_ag, stream)
    e1.record()
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / reps
    B.pl_schedule_destroy(rs)
    B.pl_schedule_destroy(ag)
    return {"ms_per_step": ms, "steps": reps, "vs_headline_step": ms / plain_ms}


def measure_all_configs(peak):
    """C1, C3 (three sizes x five algorithms), C4 (both routings), C5 (three sizes, both latency
    protocols) and the stream ceilings of the bulk-copy ring, each timed with CUDA events in this
    process.  Every entry carries its algorithmic bytes (pl_schedule_info), the fraction of the
    measured copy peak and of 8 TB/s, and the fraction of the matching stream ceiling."""
    import bench_suite as S
    from paper_2609_36954_b200 import binding as B
    b = S.Bench(quiet=True)
    streams = S.probe(b)
    ceil = {"read": streams["bulk-copy ring: read"], "write": streams["bulk-copy ring: write"],
            "copy": streams["bulk-copy ring: copy"], "mix_1r_8w": streams["bulk-copy ring: 1 read : 8 writes"]}
    out = {"stream_ceilings_gbs": {k: round(v, 1) for k, v in streams.items()}}

    def which_ceiling(read_b, write_b):
        share = read_b / max(1, read_b + write_b)
        return "read" if share >= 0.8 else "mix_1r_8w" if share <= 0.2 else "copy"

    def entry(rec, note=None):
        if rec is None or "error" in rec:
            return {"error": (rec or {}).get("error", "not built")}
        alg = rec["bytes_read"] + rec["bytes_written"]
        comp = rec["compulsory_bytes"]
        us = rec["us"] * max(1, rec["layers"])
        gbs = comp / us / 1e3
        c = which_ceiling(comp - rec["bytes_written"], rec["bytes_written"])
        e = {"us": round(rec["us"], 3), "us_p10": round(rec["us_p10"], 3), "us_p90": round(rec["us_p90"], 3),
             "message_bytes": rec["message_bytes"], "algorithmic_bytes": alg, "hbm_bytes": comp,
             "algbw_gbs": round(rec["eff_gbs"], 1), "hbm_gbs": round(gbs, 1),
             "frac_measured": round(gbs / peak, 4), "frac_8TBps": round(gbs / NOMINAL_HBM_GBS, 4),
             "ceiling": c, "frac_of_ceiling": round(gbs / ceil[c], 4),
             "grid": rec["grid"], "threads": rec["threads"], "datapath": rec["datapath"], "status": rec["status"]}
        if rec.get("us_graph128") is not None:
            e["us_in_128_call_graph"] = round(rec["us_graph128"], 3)
        if note:
            e["note"] = note
        return e

    l2 = "working set sits in L2: the HBM fractions do not apply"
    # C1: all-reduce, R = 4, 1 MiB per rank, ring, 64 KiB chunks
    out["C1"] = {name: entry(b.collective("C1", 4, dt, B.PL_ALLREDUCE, "ring", 262144, 65536, iters=50, graph=True), l2)
                 for name, dt in (("f32", B.PL_F32), ("i32", B.PL_I32))}
    # C3: all-reduce sweep points
    out["C3"] = {}
    for label, size, graph, iters in (("64KiB", 64 << 10, True, 30), ("16MiB", 16 << 20, False, 20), ("256MiB", 256 << 20, False, 8)):
        out["C3"][label] = {}
        for algo in ("ring", "tree", "oneshot", "direct", "fused"):
            chunk = max(16, min(MIB, size if (algo == "oneshot" or (algo == "tree" and size <= (128 << 10))) else size // 8))
            rec = b.collective("C3", 8, B.PL_BF16, B.PL_ALLREDUCE, algo, size // 2, chunk, iters=iters, graph=graph)
            out["C3"][label][algo] = entry(rec, l2 if size < (32 << 20) else None)
    # all-to-all and the stand-alone C2 collectives (no neighbour launch dirtying L2)
    out["C2_alone"] = {
        "reduce_scatter": entry(b.collective("C2-RS", 8, B.PL_BF16, B.PL_REDUCE_SCATTER, "direct", 32 * MIB, MIB)),
        "all_gather": entry(b.collective("C2-AG", 8, B.PL_BF16, B.PL_ALLGATHER, "direct", 4 * MIB, MIB)),
        "reduce_scatter_ring": entry(b.collective("C2-RS", 8, B.PL_BF16, B.PL_REDUCE_SCATTER, "ring", 32 * MIB, 256 << 10)),
        "all_gather_ring": entry(b.collective("C2-AG", 8, B.PL_BF16, B.PL_ALLGATHER, "ring", 4 * MIB, 256 << 10)),
        "all_to_all": entry(b.collective("A2A", 8, B.PL_BF16, B.PL_ALLTOALL, "direct", 32 * MIB, MIB)),
    }
    # the same two collectives at 256 MiB per rank: what the datapath sustains once launch, ramp and
    # tail (about 9 us per launch) stop mattering
    out["C2_alone_256MiB"] = {
        "reduce_scatter": entry(b.collective("C2-RS", 8, B.PL_BF16, B.PL_REDUCE_SCATTER, "direct", 128 * MIB, MIB, iters=10)),
        "all_gather": entry(b.collective("C2-AG", 8, B.PL_BF16, B.PL_ALLGATHER, "direct", 16 * MIB, MIB, iters=10)),
    }
    # staged schedules (ordinary application buffers), back-to-back executes without events in between:
    # one staging buffer, overlapped launches, two buffers alternated by launch parity (stage ahead)
    out["staged_back_to_back"] = {}
    for label, coll, count in (("allreduce_64MiB", B.PL_ALLREDUCE, 32 * MIB), ("reduce_scatter_64MiB", B.PL_REDUCE_SCATTER, 32 * MIB),
                               ("allreduce_1MiB", B.PL_ALLREDUCE, MIB // 2)):
        out["staged_back_to_back"][label] = {}
        for name, fl in (("one_buffer", B.PL_OPT_STAGED), ("one_buffer_overlapped_launches", B.PL_OPT_STAGED | B.PL_OPT_OVERLAP_LAUNCH),
                         ("two_buffers_stage_ahead", B.PL_OPT_STAGED | B.PL_OPT_OVERLAP_LAUNCH | B.PL_OPT_STAGE_AHEAD)):
            rec = b.collective("staged", 8, B.PL_BF16, coll, "direct", count, max(16, min(MIB, count * 2 // 8)), iters=50, back_to_back=True, flags=fl)
            out["staged_back_to_back"][label][name] = entry(rec)
    # processing phase folded into the reduce (scale, residual, fp32 output): fused all-reduce, 64 MiB per rank
    out["processing_phase"] = {}
    for name, kw in (("plain", {}), ("scale", dict(out_scale=0.125)), ("scale_residual", dict(out_scale=0.125, hook=B.PL_HOOK_RESIDUAL)),
                     ("f32_out", dict(hook=B.PL_HOOK_F32_OUT))):
        out["processing_phase"][name] = entry(b.collective("hook", 8, B.PL_BF16, B.PL_REDUCE_SCATTER, "direct", 32 * MIB, MIB, **kw))
    # the same phase on the fused all-reduce, whose results go to all 8 outputs
    for name, kw in (("fused_allreduce_plain", {}), ("fused_allreduce_scale_residual", dict(out_scale=0.125, hook=B.PL_HOOK_RESIDUAL)),
                     ("fused_allreduce_f32_out", dict(hook=B.PL_HOOK_F32_OUT))):
        out["processing_phase"][name] = entry(b.collective("hook", 8, B.PL_BF16, B.PL_ALLREDUCE, "fused", 32 * MIB, MIB, iters=10, **kw))
    # C4: MoE dispatch / combine at the full shape, both routings
    out["C4"] = {}
    for name, ident in (("permuted", False), ("identity", True)):
        r = b.moe("C4", identity=ident, dedup=False)
        out["C4"][name] = {
            "dispatch_us": round(r["dispatch_us"], 1), "combine_us": round(r["combine_us"], 1),
            "algorithmic_bytes_each": r["dispatch_bytes"], "rows": r["rows"], "max_over_mean_rows": round(r["max_over_mean_rows"], 2),
            "dispatch_hbm_gbs": round(r["dispatch_gbs"], 1), "combine_hbm_gbs": round(r["combine_gbs"], 1),
            "dispatch_frac_measured": round(r["dispatch_frac_measured"], 4), "combine_frac_measured": round(r["combine_frac_measured"], 4),
            "dispatch_frac_8TBps": round(r["dispatch_gbs"] / NOMINAL_HBM_GBS, 4), "combine_frac_8TBps": round(r["combine_gbs"] / NOMINAL_HBM_GBS, 4),
            "dispatch_frac_of_ceiling": round(r["dispatch_gbs"] / ceil["mix_1r_8w"], 4), "dispatch_ceiling": "mix_1r_8w",
            "combine_frac_of_ceiling": round(r["combine_gbs"] / ceil["read"], 4), "combine_ceiling": "read", "status": r["status"]}
    # C5: 80 layers per launch; per layer.  Flags (register executor) at the three benchmark sizes,
    # then the two latency protocols side by side at 4 / 16 / 64 KiB.
    out["C5"] = {}
    for label, count in (("16KiB", 8192), ("128KiB", 65536), ("1MiB", 524288)):
        out["C5"][label] = {algo: entry(b.collective("C5", 8, B.PL_BF16, B.PL_ALLREDUCE, algo, count, 0, iters=100, layers=80), l2)
                            for algo in ("oneshot", "fused")}
    out["C5_protocols"] = {}
    for kib in (1, 4, 16, 64):
        flags = [b.collective("C5", 8, B.PL_BF16, B.PL_ALLREDUCE, algo, kib * 512, 0, iters=200, layers=80) for algo in ("oneshot", "fused")]
        best = min(flags, key=lambda r: r["us"])
        pk = b.collective("C5", 8, B.PL_BF16, B.PL_ALLREDUCE, "oneshot", kib * 512, 0, iters=200, layers=80, datapath=B.PL_DP_PACKET)
        out["C5_protocols"]["%dKiB" % kib] = {
            "flags": {"algo": best["algo"], "p50_us": round(best["us"], 3), "p10_us": round(best["us_p10"], 3), "p90_us": round(best["us_p90"], 3), "grid": best["grid"]},
            "packets": {"algo": "oneshot", "p50_us": round(pk["us"], 3), "p10_us": round(pk["us_p10"], 3), "p90_us": round(pk["us_p90"], 3), "grid": pk["grid"]}}
    return out


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
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", default="purlin", choices=["purlin", "reference"])
    ap.add_argument("--suite", action="store_true", help="run every configuration (bench_suite.py)")
    ap.add_argument("--cpu-suite", action="store_true", help="time the CPU oracle on samples of every configuration (1 thread and all cores)")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu", action="store_true")
    ap.add_argument("--no-latency", action="store_true")
    ap.add_argument("--no-detail", action="store_true", help="skip the other configurations (C1, C3, C4, C5, stream ceilings)")
    ap.add_argument("--ag-grid", type=int, default=0, help="grid of the all-gather schedule (skips pl_comm_tune); for profiling runs")
    ap.add_argument("--ag-idle", default="", help="with --ag-grid: window of idle SMs of the all-gather launch as first:count")
    ap.add_argument("--no-tune", action="store_true", help="skip pl_comm_tune (the all-gather then runs with the untuned default grid)")
    ap.add_argument("--plain-options", action="store_true", help="build the two schedules of the step without PL_OPT_INPUTS_LAST_USE")
    ap.add_argument("--min-timed-ms", type=float, default=500.0, help="repeat the K-step block until the timed region lasts this long")
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
    ap.add_argument("--replica-selftest", action="store_true",
                    help="only join the process group (gloo), take a barrier and a max over ranks, print one line: "
                         "checks the multi-process plumbing without a GPU")
    args = ap.parse_args()
    # --gpus N: N independent replicas, one process per GPU.  Under a launcher (torchrun) the
    # environment describes the group and must agree with --gpus; without one, this process starts
    # the N replicas itself.
    env_world = os.environ.get("WORLD_SIZE")
    if env_world is not None and int(env_world) != args.gpus and args.impl != "reference":
        raise SystemExit(f"bench.py: --gpus {args.gpus} disagrees with WORLD_SIZE={env_world} of the launcher")
    if env_world is None and args.gpus > 1 and args.impl != "reference" and not args.cpu_suite and not args.suite:
        from paper_2609_36954_b200 import replicas
        raise SystemExit(replicas.launch_local(args.gpus, [sys.executable, os.path.abspath(__file__)] + sys.argv[1:]))
    if args.replica_selftest:
        from paper_2609_36954_b200 import replicas
        n, rank, _ = replicas.init("gloo")
        replicas.barrier()
        slow = replicas.max_over_ranks(1.0 + rank)
        replicas.barrier()
        if rank == 0:
            print(json.dumps({"selftest": True, "n_gpus": n, "max_over_ranks": slow}))
        replicas.finalize()
        return
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
