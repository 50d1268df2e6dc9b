#!/usr/bin/env python
"""Turns the JSON line printed by ``bench.py`` into the markdown tables of the design notes.

  python bench.py > line.json
  python bench_table.py line.json

Nothing is measured here: every number is read from the line (its ``detail`` section holds one
entry per configuration, each with its algorithmic bytes and fractions).
"""
from __future__ import annotations

import json
import sys


def f(x, nd=1):
    return "-" if x is None else f"{x:.{nd}f}"


def row(cells):
    return "| " + " | ".join(str(c) for c in cells) + " |"


def collective_rows(name, e):
    if "error" in e:
        return row([name, e["error"]] + [""] * 7)
    return row([name, f(e["us"], 2) + (f" ({f(e['us_in_128_call_graph'], 2)} in a 128-call graph)" if "us_in_128_call_graph" in e else ""),
                f(e["algorithmic_bytes"] / 2 ** 20, 1), f(e["hbm_bytes"] / 2 ** 20, 1), f(e["algbw_gbs"], 0), f(e["hbm_gbs"], 0),
                f(e["frac_measured"], 3), f(e["frac_8TBps"], 3), f"{f(e['frac_of_ceiling'], 3)} ({e['ceiling']})"])


def main(path):
    with open(path) as fh:
        line = json.loads([l for l in fh.read().splitlines() if l.startswith("{")][-1])
    d = line["detail"]
    print(f"Headline: {f(line['value'], 1)} {line['unit']} effective, {f(line['ms_per_step'] * 1e3, 1)} us per step "
          f"({d['timed_region']['blocks']} blocks of {d['timed_region']['steps_per_block']} steps, median block); "
          f"reduce-scatter launch {f(d['reduce_scatter']['us'], 1)} us = {f(d['reduce_scatter']['hbm_gbs'], 0)} GB/s "
          f"({f(d['reduce_scatter']['frac_measured'], 3)} of measured, {f(d['reduce_scatter']['frac_8TBps'], 3)} of 8 TB/s), "
          f"all-gather launch {f(d['all_gather']['us'], 1)} us ({f(d['all_gather']['frac_measured'], 3)} of measured on compulsory bytes); "
          f"end to end {f(line['e2e']['value'], 2)} GB/s; clocks {line['clocks']['sm_mhz']} MHz {line['clocks']['reasons']}.")
    if "step_both_launches_overlapped" in d:
        o = d["step_both_launches_overlapped"]
        print(f"Step with both launches overlapped: {f(o['ms_per_step'] * 1e3, 1)} us ({f(o['vs_headline_step'], 3)} of the headline step).")
    if "step_without_last_use_hint" in d:
        o = d["step_without_last_use_hint"]
        print(f"Step without PL_OPT_INPUTS_LAST_USE: {f(o['ms_per_step'] * 1e3, 1)} us ({f(o['vs_headline_step'], 3)} of the headline step).")
    r = line["roofline"]
    if "traffic_in_situ" in r:
        print(f"Reduce-scatter DRAM traffic per launch: {f(r['traffic'] / 1e6, 1)} MB captured alone, {f(r['traffic_in_situ'] / 1e6, 1)} MB inside the step "
              f"({f(r['dram_gbs_in_situ'], 0)} GB/s of DRAM traffic in situ).")
    c = d.get("configs")
    if not c:
        return
    print("\nStream ceilings (GB/s): " + ", ".join(f"{k} {v:.0f}" for k, v in c["stream_ceilings_gbs"].items()))
    head = ["configuration", "us", "algorithmic MiB", "HBM MiB", "algbw GB/s", "HBM GB/s", "of measured", "of 8 TB/s", "of stream ceiling"]
    print("\n" + row(head) + "\n" + row(["---"] * len(head)))
    for k, e in c["C1"].items():
        print(collective_rows(f"C1 ring all-reduce R=4 1 MiB {k}", e))
    for k, e in c["C2_alone"].items():
        print(collective_rows(f"C2 {k} alone, 64 MiB", e))
    for k, e in c.get("C2_alone_256MiB", {}).items():
        print(collective_rows(f"C2 {k} alone, 256 MiB", e))
    for size, algos in c["C3"].items():
        for k, e in algos.items():
            print(collective_rows(f"C3 all-reduce {size} {k}", e))
    for k, e in c["C5"].items():
        for a, ee in e.items():
            print(collective_rows(f"C5 80 layers x {k} {a} (per layer)", ee))
    for k, e in c.get("staged_back_to_back", {}).items():
        for a, ee in e.items():
            print(collective_rows(f"staged {k} {a}", ee))
    for k, e in c.get("processing_phase", {}).items():
        what = "fused all-reduce" if k.startswith("fused_allreduce_") else "reduce-scatter"
        print(collective_rows(f"{what} 64 MiB, processing phase: {k.replace('fused_allreduce_', '')}", e))
    print("\n" + row(["C4 routing", "dispatch us", "of measured", "of 8 TB/s", "of 1:8 ceiling", "combine us", "of measured", "of 8 TB/s", "of read ceiling"]))
    print(row(["---"] * 9))
    for k, e in c["C4"].items():
        print(row([k, e["dispatch_us"], e["dispatch_frac_measured"], e["dispatch_frac_8TBps"], e["dispatch_frac_of_ceiling"],
                   e["combine_us"], e["combine_frac_measured"], e["combine_frac_8TBps"], e["combine_frac_of_ceiling"]]))
    print("\n" + row(["latency protocol, per layer", "flags p50 / p10 / p90 us", "packets p50 / p10 / p90 us"]))
    print(row(["---"] * 3))
    for k, e in c["C5_protocols"].items():
        fl, pk = e["flags"], e["packets"]
        print(row([k, f"{fl['p50_us']} / {fl['p10_us']} / {fl['p90_us']} ({fl['algo']}, grid {fl['grid']})",
                   f"{pk['p50_us']} / {pk['p10_us']} / {pk['p90_us']} (grid {pk['grid']})"]))


if __name__ == "__main__":
    main(sys.argv[1])
