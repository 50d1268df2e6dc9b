"""Timing of every benchmark configuration on one GPU (CUDA events, C-ABI calls only).

Used by ``bench.py --suite``.  One JSON line per measured point:
effective GB/s (message size / time, the paper's algorithm bandwidth), schedule GB/s
(bytes the schedule reads + writes / time), fraction of the HBM peak, and microseconds.
Inputs are seeded synthetic data of the configuration's shape; values do not influence
timing, so large buffers are filled by tiling a generated block.
"""
from __future__ import annotations

import json
import os
import sys

import numpy as np
import torch

from paper_2609_36954_b200 import binding as B
from paper_2609_36954_b200 import inputs as gen

MIB = 1 << 20
ALGO = {"ring": B.PL_ALGO_RING, "tree": B.PL_ALGO_TREE, "direct": B.PL_ALGO_DIRECT,
        "oneshot": B.PL_ALGO_ONESHOT, "fused": B.PL_ALGO_DIRECT_FUSED}


def _peak():
    root = os.path.dirname(os.path.abspath(__file__))
    try:
        return float(json.load(open(os.path.join(root, "MEASURED_PEAKS.json")))["hbm_gbs"])
    except Exception:
        return 6650.0


def _fill(nbytes, stream_id):
    """Device buffer of nbytes filled with tiled bf16 N(0,1) bits."""
    blk = gen.normal_bf16(min(nbytes // 2, 1 << 20) or 8, 0, stream_id)
    t = torch.from_numpy(blk.view(np.int16)).cuda()
    reps = (nbytes // 2 + t.numel() - 1) // t.numel()
    return t.repeat(reps)[: max(8, nbytes // 2)].contiguous()


def _time(fn, iters, warmup=3, per_call_events=False):
    iters = int(os.environ.get("PL_SUITE_ITERS", iters))  # short runs for profiler captures
    for _ in range(warmup):
        fn()
    torch.cuda.synchronize()
    if per_call_events:
        ev = [torch.cuda.Event(enable_timing=True) for _ in range(iters + 1)]
        ev[0].record()
        for i in range(iters):
            fn()
            ev[i + 1].record()
        torch.cuda.synchronize()
        ms = np.array([ev[i].elapsed_time(ev[i + 1]) for i in range(iters)])
        return float(np.median(ms) * 1e3), float(np.percentile(ms, 10) * 1e3), float(np.percentile(ms, 90) * 1e3)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(iters):
        fn()
    e1.record()
    torch.cuda.synchronize()
    us = e0.elapsed_time(e1) * 1e3 / iters
    return us, us, us


def _time_graph(launch, calls=128, replays=8):
    """The paper's microbenchmark method (Sec. 5): capture `calls` invocations in a CUDA graph,
    replay once to warm up, time `replays` replays with CUDA events, divide by calls*replays.
    `launch(stream_handle)` must enqueue exactly one invocation on the given stream."""
    g = torch.cuda.CUDAGraph()
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.graph(g, stream=side):
        h = torch.cuda.current_stream().cuda_stream
        for _ in range(calls):
            launch(h)
    g.replay()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(replays):
        g.replay()
    e1.record()
    torch.cuda.synchronize()
    return e0.elapsed_time(e1) * 1e3 / (calls * replays)


class Bench:
    def __init__(self, out_path=None, opts_kw=None, quiet=False):
        self.peak = _peak()
        self.out = open(out_path, "w") if out_path else None
        self.stream = torch.cuda.current_stream().cuda_stream
        self.opts_kw = opts_kw or {}
        self.quiet = quiet       # collect the records instead of printing them (bench.py's detail section)
        self.records = []

    def emit(self, rec):
        self.records.append(rec)
        if self.quiet:
            return
        line = json.dumps(rec)
        print(line, flush=True)
        if self.out:
            self.out.write(line + "\n")
            self.out.flush()

    def collective(self, cfg, R, dtype, coll, algo, count, chunk, iters=20, layers=0, graph=False, root=None,
                   back_to_back=False, **kw):
        comm = B.pl_comm_create(R, dtype)
        okw = dict(self.opts_kw)
        okw.update(kw)
        opts = B.make_opts(**okw)
        try:
            if root is not None:
                s = B.pl_schedule_build_rooted(comm, coll, root, count, chunk, opts)
            elif layers:
                s = B.pl_schedule_build_layers(comm, ALGO[algo], count, layers, opts)
            else:
                s = B.pl_schedule_build(comm, coll, ALGO[algo], count, chunk, opts)
        except B.PurlinError as e:
            B.pl_comm_destroy(comm)
            self.emit({"cfg": cfg, "algo": algo, "error": str(e)})
            return None
        info = B.pl_schedule_info(s)
        d_in = [_fill(int(info.in_bytes[r]), r) for r in range(R)]
        d_out = [torch.empty(max(16, int(info.out_bytes[r])), dtype=torch.uint8, device="cuda") for r in range(R)]
        d_aux = [_fill(int(info.aux_bytes[r]), 100 + r) for r in range(R)] if any(info.aux_bytes[r] for r in range(R)) else None
        bufs = B.make_bufs([t.data_ptr() for t in d_in], [t.data_ptr() for t in d_out],
                           [int(info.in_bytes[r]) for r in range(R)], [int(info.out_bytes[r]) for r in range(R)],
                           [t.data_ptr() for t in d_aux] if d_aux else None, [int(info.aux_bytes[r]) for r in range(R)] if d_aux else None)
        # back_to_back: no event between the launches, so that overlapped launches can overlap
        p50, p10, p90 = _time(lambda: B.pl_execute(s, bufs, self.stream), iters, per_call_events=not back_to_back)
        graph_us = None
        if graph:
            graph_us = _time_graph(lambda h: B.pl_execute(s, bufs, h)) / max(1, layers)
        st = B.pl_comm_status(comm)
        in_kernel = None
        if layers and (okw.get("flags", 0) & B.PL_OPT_TRACE):
            # per-layer latency from the in-kernel stamps of the last execute: a layer is
            # complete when the last of its signalling ops is about to release its flag
            ops = B.pl_schedule_dump(s)
            tr = B.pl_schedule_trace_read(s, len(ops), self.stream)
            done = np.zeros(layers, dtype=np.float64)
            for o in ops:
                done[o.layer] = max(done[o.layer], float(tr[o.topo, 1]), float(tr[o.topo, 0]))
            gaps = np.diff(done[:-1]) / 1e3  # the last layer's ops do not signal
            in_kernel = {"p50_us": float(np.median(gaps)), "p10_us": float(np.percentile(gaps, 10)),
                         "p90_us": float(np.percentile(gaps, 90))}
        nl = max(1, layers)
        sched_bytes = info.bytes_read + info.bytes_written
        # bytes that must cross the HBM interface when nothing is cached between launches
        # (pl_sched_info_t.hbm_bytes: input bytes once however often they are read, everything else as scheduled)
        rec = {"cfg": cfg, "bytes_read": int(info.bytes_read), "bytes_written": int(info.bytes_written),
               "compulsory_bytes": int(info.hbm_bytes), "coll": int(coll), "algo": algo, "R": R, "dtype": int(dtype),
               "message_bytes": int(info.message_bytes), "chunk": int(min(chunk, 1 << 40)), "layers": layers,
               "us": p50 / nl, "us_p10": p10 / nl, "us_p90": p90 / nl, "us_graph128": graph_us, "layer_us_in_kernel": in_kernel,
               "eff_gbs": info.message_bytes * nl / p50 / 1e3, "sched_gbs": sched_bytes / p50 / 1e3,
               "hbm_frac_measured": sched_bytes / p50 / 1e3 / self.peak, "hbm_frac_8TBps": sched_bytes / p50 / 1e3 / 8000.0,
               "n_ops": int(info.n_ops), "grid": int(info.grid), "threads": int(info.threads),
               "slice_bytes": int(info.slice_bytes), "datapath": int(info.datapath), "status": int(st.code)}
        self.emit(rec)
        B.pl_schedule_destroy(s)
        B.pl_comm_destroy(comm)
        del d_in, d_out
        return rec

    def collective_v(self, cfg, R, dtype, coll, counts, chunk, iters=20, **kw):
        """Variable-size collectives (counts as pl_schedule_build_v takes them)."""
        comm = B.pl_comm_create(R, dtype)
        s = B.pl_schedule_build_v(comm, coll, B.PL_ALGO_DIRECT, counts, chunk, B.make_opts(**kw))
        info = B.pl_schedule_info(s)
        d_in = [_fill(int(info.in_bytes[r]), r) for r in range(R)]
        d_out = [torch.empty(max(16, int(info.out_bytes[r])), dtype=torch.uint8, device="cuda") for r in range(R)]
        bufs = B.make_bufs([t.data_ptr() for t in d_in], [t.data_ptr() for t in d_out],
                           [int(info.in_bytes[r]) for r in range(R)], [int(info.out_bytes[r]) for r in range(R)])
        p50, _, _ = _time(lambda: B.pl_execute(s, bufs, self.stream), iters, per_call_events=True)
        graph_us = _time_graph(lambda h: B.pl_execute(s, bufs, h)) if info.message_bytes <= 2 * MIB else None
        sched_bytes = info.bytes_read + info.bytes_written
        self.emit({"cfg": cfg, "coll": int(coll), "algo": "direct", "R": R, "message_bytes": int(info.message_bytes),
                   "us": p50, "us_graph128": graph_us, "eff_gbs": info.message_bytes / p50 / 1e3,
                   "sched_gbs": sched_bytes / p50 / 1e3, "hbm_frac_measured": sched_bytes / p50 / 1e3 / self.peak,
                   "n_ops": int(info.n_ops), "grid": int(info.grid), "datapath": int(info.datapath),
                   "status": int(B.pl_comm_status(comm).code)})
        B.pl_schedule_destroy(s)
        B.pl_comm_destroy(comm)

    def moe(self, cfg, R=8, T=4096, H=7168, E=256, K=8, identity=False, iters=10, dedup=True):
        idx, gates = gen.moe_routing(R, T, E, K, identity_perm=identity)
        counts = np.zeros((R, R), np.int64)
        for p in range(R):
            counts[p] = np.bincount(idx[p].ravel() // (E // R), minlength=R)
        cap = int(counts.sum(axis=0).max())
        comm = B.pl_comm_create(R, B.PL_BF16)
        plan = B.pl_moe_plan_create(comm, T, H, E, K, cap)
        d_x = [_fill(T * H * 2, r) for r in range(R)]
        d_i = [torch.from_numpy(a).cuda() for a in idx]
        d_g = [torch.from_numpy(a).cuda() for a in gates]
        d_recv = [torch.empty(cap * H, dtype=torch.int16, device="cuda") for _ in range(R)]
        d_meta = [torch.empty(cap * 4, dtype=torch.int32, device="cuda") for _ in range(R)]
        d_out = [torch.empty(T * H, dtype=torch.int16, device="cuda") for _ in range(R)]
        px = [t.data_ptr() for t in d_x]
        pi = [t.data_ptr() for t in d_i]
        pr = [t.data_ptr() for t in d_recv]
        pm = [t.data_ptr() for t in d_meta]
        pg = [t.data_ptr() for t in d_g]
        po = [t.data_ptr() for t in d_out]
        disp, _, _ = _time(lambda: B.pl_moe_dispatch(plan, px, pi, pr, pm, self.stream), iters, per_call_events=True)
        comb, _, _ = _time(lambda: B.pl_moe_combine(plan, pr, pg, po, self.stream), iters, per_call_events=True)
        st = B.pl_moe_plan_read(plan, 0, 0, 0, self.stream)
        rows = R * T * K
        row_b = H * 2
        d_bytes = R * T * row_b + rows * row_b
        c_bytes = rows * row_b + R * T * row_b
        rec = {"cfg": cfg, "routing": "identity" if identity else "permuted", "rows": rows, "cap": cap,
               "max_over_mean_rows": float(counts.sum(axis=0).max() / counts.sum(axis=0).mean()),
               "dispatch_us": disp, "combine_us": comb, "dispatch_bytes": d_bytes, "combine_bytes": c_bytes,
               "dispatch_gbs": d_bytes / disp / 1e3, "combine_gbs": c_bytes / comb / 1e3,
               "dispatch_frac_measured": d_bytes / disp / 1e3 / self.peak,
               "combine_frac_measured": c_bytes / comb / 1e3 / self.peak, "status": int(st)}
        if dedup:
            # deduplicated variant on the same plan: one row per (token, destination rank)
            dd, _, _ = _time(lambda: B.pl_moe_dispatch_dedup(plan, px, pi, pr, pm, self.stream), iters, per_call_events=True)
            dc, _, _ = _time(lambda: B.pl_moe_combine_dedup(plan, pr, po, self.stream), iters, per_call_events=True)
            cnt = np.zeros((R, R), np.int64)
            B.pl_moe_plan_read_dedup(plan, 0, cnt.ctypes.data, self.stream)
            rows_dd = int(cnt.sum())
            rec.update({"dedup_rows": rows_dd, "dedup_dispatch_us": dd, "dedup_combine_us": dc,
                        "dedup_dispatch_gbs": (R * T + rows_dd) * H * 2 / dd / 1e3,
                        "dedup_combine_gbs": (R * T + rows_dd) * H * 2 / dc / 1e3})
        self.emit(rec)
        B.pl_moe_plan_destroy(plan)
        B.pl_comm_destroy(comm)
        return rec


def probe(b):
    """Reference points from library kernels on the same GPU (context for the roofline
    fractions, not part of the product path): plain copy, fill and read over 1 GiB.  Returns
    {stream name: GB/s}."""
    n = 1 << 30
    found = {}
    a = torch.empty(n, dtype=torch.uint8, device="cuda")
    c = torch.empty(n, dtype=torch.uint8, device="cuda")
    a.zero_()
    c.zero_()
    af = a.view(torch.float32)
    for name, fn, nbytes in (("torch copy_ (read+write)", lambda: c.copy_(a), 2 * n),
                             ("torch fill_ (write)", lambda: a.fill_(1), n),
                             ("torch sum fp32 (read)", lambda: af.sum(), n)):
        us, _, _ = _time(fn, 20)
        b.emit({"cfg": "probe", "what": name, "gbs": nbytes / us / 1e3})
        found[name] = nbytes / us / 1e3
    # the same three streams through the library's own bulk-copy ring (pl_probe_hbm)
    h = torch.cuda.current_stream().cuda_stream
    for name, kind, nbytes in (("bulk-copy ring: read", 0, n), ("bulk-copy ring: write", 1, n), ("bulk-copy ring: copy", 2, 2 * n)):
        us, _, _ = _time(lambda: B.pl_probe_hbm(kind, a.data_ptr(), c.data_ptr(), n, 0, h), 20)
        b.emit({"cfg": "probe", "what": name, "gbs": nbytes / us / 1e3})
        found[name] = nbytes / us / 1e3
    # one read to eight writes (the mix of the all-gather and of the MoE dispatch): 128 MiB in, 1 GiB out
    m = n // 8
    us, _, _ = _time(lambda: B.pl_probe_hbm(3, a.data_ptr(), c.data_ptr(), m, 0, h), 20)
    b.emit({"cfg": "probe", "what": "bulk-copy ring: 1 read : 8 writes", "gbs": 9 * m / us / 1e3})
    found["bulk-copy ring: 1 read : 8 writes"] = 9 * m / us / 1e3
    return found


def main(args=None):
    which = os.environ.get("PL_SUITE", "probe,c1,c2,a2a,staged,varlen,rooted,c3,c4,c5").split(",")
    out = os.environ.get("PL_SUITE_OUT")  # optional file that receives the JSON lines too
    if out and os.path.dirname(out):
        os.makedirs(os.path.dirname(out), exist_ok=True)
    b = Bench(out)
    if "probe" in which:
        probe(b)
    if "c1" in which:
        for dt in (B.PL_F32, B.PL_I32):
            b.collective("C1", 4, dt, B.PL_ALLREDUCE, "ring", 262144, 65536, iters=50, graph=True)
    if "c2" in which:
        n = 32 * MIB  # 64 MiB bf16 per rank
        for algo in ("direct", "ring"):
            for chunk in (256 * 1024, MIB):
                b.collective("C2-RS", 8, B.PL_BF16, B.PL_REDUCE_SCATTER, algo, n, chunk)
                b.collective("C2-AG", 8, B.PL_BF16, B.PL_ALLGATHER, algo, n // 8, chunk)
    if "c2big" in which:
        # the same two collectives at 256 MiB per rank: the sustained rate, launch edges amortised
        n = 128 * MIB
        b.collective("C2-RS-256MiB", 8, B.PL_BF16, B.PL_REDUCE_SCATTER, "direct", n, MIB, iters=10)
        b.collective("C2-AG-256MiB", 8, B.PL_BF16, B.PL_ALLGATHER, "direct", n // 8, MIB, iters=10)
    if "staged" in which:
        # the paper's default setting: ordinary application buffers, so the work of staging is
        # included (Sec. 5, "Collective Microbenchmarks"); full and restricted staging capacity
        n = 32 * MIB
        for cap in (0, 32 * MIB):
            kw = dict(flags=B.PL_OPT_STAGED, staging_bytes=cap)
            b.collective("staged-RS cap=%d" % cap, 8, B.PL_BF16, B.PL_REDUCE_SCATTER, "direct", n, MIB, **kw)
            b.collective("staged-AG cap=%d" % cap, 8, B.PL_BF16, B.PL_ALLGATHER, "direct", n // 8, MIB,
                         flags=B.PL_OPT_STAGED, staging_bytes=cap // 8)
            b.collective("staged-A2A cap=%d" % cap, 8, B.PL_BF16, B.PL_ALLTOALL, "direct", n, MIB, **kw)
            for size in (MIB, 16 * MIB, 64 * MIB, 256 * MIB):
                b.collective("staged-AR cap=%d" % cap, 8, B.PL_BF16, B.PL_ALLREDUCE, "direct", size // 2,
                             max(16, min(MIB, size // 8)), iters=10, **kw)
    if "stage_ahead" in which:
        # back-to-back staged executes: one staging buffer, overlapped launches, and two staging
        # buffers alternated by launch parity with the stage role running ahead (Sec. 4.1-4.2)
        for name, coll, count in (("AR", B.PL_ALLREDUCE, 32 * MIB), ("RS", B.PL_REDUCE_SCATTER, 32 * MIB), ("AR-1MiB", B.PL_ALLREDUCE, MIB // 2),
                                  ("AR-16MiB", B.PL_ALLREDUCE, 8 * MIB)):
            for label, fl in (("one buffer", B.PL_OPT_STAGED), ("one buffer, overlapped launches", B.PL_OPT_STAGED | B.PL_OPT_OVERLAP_LAUNCH),
                              ("two buffers, stage ahead", B.PL_OPT_STAGED | B.PL_OPT_OVERLAP_LAUNCH | B.PL_OPT_STAGE_AHEAD)):
                b.collective("staged-%s %s" % (name, label), 8, B.PL_BF16, coll, "direct", count, max(16, min(MIB, count * 2 // 8)), iters=50,
                             back_to_back=True, flags=fl)
    if "rooted" in which:
        for size in (64 * 1024, 64 * MIB):
            for name, coll, count in (("broadcast", B.PL_BROADCAST, size // 2), ("reduce", B.PL_REDUCE, size // 2),
                                      ("scatter", B.PL_SCATTER, size // 16), ("gather", B.PL_GATHER, size // 16)):
                b.collective("rooted-" + name, 8, B.PL_BF16, coll, "direct", count, MIB, root=0, graph=size < MIB)
    if "a2a" in which:
        # all-to-all: a pure copy, every byte read once from HBM and written once (64 MiB per rank first:
        # the case the profiler summary under profiles/ captures)
        for mib in (64, 16, 256):
            b.collective("A2A", 8, B.PL_BF16, B.PL_ALLTOALL, "direct", mib * MIB // 2, MIB)
        # slice size of the copy ops: the cost model's coarse slices against the 32 KiB sweep
        for sl in (262144, 131072, 65536, 32768, 16384):
            b.collective(f"A2A-slice{sl >> 10}K", 8, B.PL_BF16, B.PL_ALLTOALL, "direct", 32 * MIB, MIB, slice_bytes=sl)
    if "ablation" in which:
        # (a) pipeline depth at a fixed CTA count: the analogue of the paper's copy ablation
        #     (Sec. 5, "ablation": bandwidth vs. number of stages S at fixed stage size)
        n = 32 * MIB
        for sb in (16384, 32768):
            for S in (2, 3, 4, 6, 8):
                if 1024 + S * sb > 227 * 1024:
                    continue
                kw = dict(datapath=B.PL_DP_TMA, stages=S, stage_bytes=sb, n_ctas=144, slice_bytes=262144)
                b.collective("depth-copy S=%d B=%d" % (S, sb), 8, B.PL_BF16, B.PL_ALLGATHER, "direct", n // 8, MIB, **kw)
                b.collective("depth-reduce S=%d B=%d" % (S, sb), 8, B.PL_BF16, B.PL_REDUCE_SCATTER, "direct", n, MIB, **kw)
        # (b) CTA count at the default ring: the analogue of the paper's SM sweep (Sec. 2.2, Fig. 2)
        for nct in (8, 16, 32, 64, 96, 128, 144):
            kw = dict(datapath=B.PL_DP_TMA, n_ctas=nct, slice_bytes=65536)
            b.collective("ctas-copy n=%d" % nct, 8, B.PL_BF16, B.PL_ALLGATHER, "direct", n // 8, MIB, **kw)
            b.collective("ctas-reduce n=%d" % nct, 8, B.PL_BF16, B.PL_REDUCE_SCATTER, "direct", n, MIB, **kw)
        # (c) register path vs bulk-copy ring on the same schedules
        for dp, name in ((B.PL_DP_LDST, "ldst"), (B.PL_DP_TMA, "tma")):
            b.collective("datapath-copy " + name, 8, B.PL_BF16, B.PL_ALLGATHER, "direct", n // 8, MIB, datapath=dp)
            b.collective("datapath-reduce " + name, 8, B.PL_BF16, B.PL_REDUCE_SCATTER, "direct", n, MIB, datapath=dp)
            b.collective("datapath-a2a " + name, 8, B.PL_BF16, B.PL_ALLTOALL, "direct", n, MIB, datapath=dp)
    if "varlen" in which:
        # the paper's variable-length workload (Appendix C): Zipf(s=0.125) split of T bytes over
        # 8 ranks; all-to-all-v rotates the split per rank so every rank sends and receives T
        for T in (64 * 1024, MIB, 64 * MIB, 1024 * MIB):
            n = (gen.zipf_split(T) // 2).tolist()
            b.collective_v("AGV", 8, B.PL_BF16, B.PL_ALLGATHERV, n, MIB)
            b.collective_v("RSV", 8, B.PL_BF16, B.PL_REDUCE_SCATTERV, n, MIB)
            if T <= 256 * MIB:
                b.collective_v("A2AV", 8, B.PL_BF16, B.PL_ALLTOALLV, (gen.alltoallv_counts_bytes(T) // 2).tolist(), MIB)
    if "c3" in which:
        for lg in range(12, 29):
            size = 1 << lg
            for algo in ("ring", "tree", "oneshot", "direct", "fused"):
                if algo == "oneshot" and size > 64 * MIB:
                    continue
                # chunks of a partition (size / 8) for the partitioned algorithms and for trees above
                # 128 KiB (a tree pipelines its levels over the chunks: 1 MiB in one chunk takes
                # 51 us, in eight 23 us), of the whole message for one-shot and small trees
                chunk = max(16, min(MIB, size if (algo == "oneshot" or (algo == "tree" and size <= (128 << 10))) else size // 8))
                b.collective("C3", 8, B.PL_BF16, B.PL_ALLREDUCE, algo, size // 2, chunk, iters=30 if lg < 24 else 10,
                             graph=lg <= 24)
                # latency-bound sizes again with overlapped launches (CTAs of call i+1 set up while call i drains)
                if lg <= 20 and algo in ("oneshot", "fused"):
                    b.collective("C3-overlap", 8, B.PL_BF16, B.PL_ALLREDUCE, algo, size // 2, chunk, iters=30, graph=True,
                                 flags=B.PL_OPT_OVERLAP_LAUNCH)
    if "c4" in which:
        T = int(os.environ.get("PL_MOE_TOKENS", 4096))  # fewer tokens per rank for profiler captures
        b.moe("C4", T=T, identity=False)
        b.moe("C4", T=T, identity=True)
    if "c5" in which:
        for batch in (1, 8, 64):
            for algo in ("oneshot", "direct", "fused"):
                b.collective("C5", 8, B.PL_BF16, B.PL_ALLREDUCE, algo, batch * 8192, 0, iters=50, layers=80)
    if "c5prof" in which:
        # the three latency-path kernels at 16 KiB, one after the other (short: for profiler captures)
        b.collective("C5-flags", 8, B.PL_BF16, B.PL_ALLREDUCE, "fused", 8192, 0, iters=20, layers=80)
        b.collective("C5-flags", 8, B.PL_BF16, B.PL_ALLREDUCE, "oneshot", 8192, 0, iters=20, layers=80)
        b.collective("C5-packets", 8, B.PL_BF16, B.PL_ALLREDUCE, "oneshot", 8192, 0, iters=20, layers=80, datapath=B.PL_DP_PACKET)
    if "c5trace" in which:
        # where a layer's time goes, from the in-kernel stamps of the last execute (PL_OPT_TRACE): for
        # every op "start" = its waits are satisfied (flags seen / one packet of every rank seen) and
        # "end" = its output is written and it is about to signal (flags) or to join its rank (packets)
        for kib in (4, 16):
            for name, algo, kw in (("flags fused", "fused", {}), ("flags oneshot", "oneshot", {}),
                                   ("packets", "oneshot", dict(datapath=B.PL_DP_PACKET))):
                comm = B.pl_comm_create(8, B.PL_BF16)
                sched = B.pl_schedule_build_layers(comm, ALGO[algo], kib * 512, 80, B.make_opts(flags=B.PL_OPT_TRACE, **kw))
                info = B.pl_schedule_info(sched)
                d_in = [_fill(int(info.in_bytes[r]), r) for r in range(8)]
                d_out = [torch.empty(int(info.out_bytes[r]), dtype=torch.uint8, device="cuda") for r in range(8)]
                bufs = B.make_bufs([t.data_ptr() for t in d_in], [t.data_ptr() for t in d_out],
                                   [int(info.in_bytes[r]) for r in range(8)], [int(info.out_bytes[r]) for r in range(8)])
                for _ in range(5):
                    B.pl_execute(sched, bufs, b.stream)
                ops = B.pl_schedule_dump(sched)
                tr = B.pl_schedule_trace_read(sched, len(ops), b.stream).astype(np.int64)
                lay = np.array([o.layer for o in ops])
                start = np.array([tr[lay == l, 0].max() for l in range(80)])   # the last op of the layer to see its inputs
                first = np.array([tr[lay == l, 0].min() for l in range(80)])
                end = np.array([tr[lay == l, 1].max() for l in range(79)])      # the last op of the layer to finish writing
                b.emit({"cfg": "C5-trace", "protocol": name, "message_bytes": kib * 1024, "grid": int(info.grid),
                        "layer_ns_p50": float(np.median(np.diff(start)[5:])),
                        "written_to_next_seen_ns_p50": float(np.median((start[1:] - end)[5:])),
                        "written_to_first_seen_ns_p50": float(np.median((first[1:] - end)[5:])),
                        "seen_to_written_ns_p50": float(np.median((end - start[:-1])[5:]))})
                B.pl_schedule_destroy(sched)
                B.pl_comm_destroy(comm)
    if "c5p" in which or "c5" in which:
        # the two latency protocols side by side: per-rank flags (register executor) against
        # 16-byte packets (8 B payload + 8 B tag), per layer, 80 layers in one launch
        for kib in (4, 16, 64):
            b.collective("C5-flags", 8, B.PL_BF16, B.PL_ALLREDUCE, "oneshot", kib * 512, 0, iters=100, layers=80)
            b.collective("C5-flags", 8, B.PL_BF16, B.PL_ALLREDUCE, "fused", kib * 512, 0, iters=100, layers=80)
            for g in (8, 4, 2, 1):
                if kib * 1024 // 16 // g <= 1024:  # at most 4 vectors per thread
                    b.collective("C5-packets G=%d" % g, 8, B.PL_BF16, B.PL_ALLREDUCE, "oneshot", kib * 512, 0, iters=100, layers=80,
                                 datapath=B.PL_DP_PACKET, n_ctas=8 * g)
    if "c5" in which:
        # the same with in-kernel time stamps: distribution of the per-layer latency inside one launch
        for batch in (1, 8, 64):
            b.collective("C5-trace", 8, B.PL_BF16, B.PL_ALLREDUCE, "fused", batch * 8192, 0, iters=20, layers=80,
                         flags=B.PL_OPT_TRACE)


if __name__ == "__main__":
    main()
