"""Turns an Nsight Compute report into the short text summary kept under ``profiles/`` and
records the DRAM traffic per element that ``bench.py`` prints as ``roofline.traffic``.

    python -m paper_2604_19906_b200.profile_summary REPORT.ncu-rep --kernel REGEX
        [--workload KEY --elements E]      # also update profiles/dram_traffic.json
        [--out profiles/NAME.md --command "the command that produced the report"]

The JSON entry stores, beside the bytes per element, a digest of the kernel sources (csrc/*.cuh) at the
time of the capture; ``bench.py`` reports ``traffic: null`` once the sources have changed.
``ncu`` must be on PATH (it reads reports without a GPU).
"""
from __future__ import annotations

import argparse
import csv
import glob
import hashlib
import json
import os
import re
import subprocess
import sys

PKG = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(PKG)
TRAFFIC_JSON = os.path.join(ROOT, "profiles", "dram_traffic.json")

METRICS = [
    "gpu__time_duration.sum", "dram__bytes_read.sum", "dram__bytes_write.sum",
    "gpu__dram_throughput.avg.pct_of_peak_sustained_elapsed",
    "sm__pipe_tensor_subpipe_dmma_cycles_active.avg.pct_of_peak_sustained_active",
    "sm__pipe_tensor_cycles_active.avg.pct_of_peak_sustained_active",
    "sm__pipe_fp64_cycles_active.avg.pct_of_peak_sustained_active",
    "sm__warps_active.avg.pct_of_peak_sustained_active",
    "launch__registers_per_thread", "launch__grid_size", "launch__block_size",
    "launch__shared_mem_per_block_dynamic",
    "l1tex__data_pipe_lsu_wavefronts_mem_shared.sum",
    "l1tex__data_bank_conflicts_pipe_lsu_mem_shared.sum",
    "l1tex__data_pipe_lsu_wavefronts_mem_shared.sum.pct_of_peak_sustained_elapsed",
    "l1tex__throughput.avg.pct_of_peak_sustained_elapsed",
    "smsp__issue_active.avg.pct_of_peak_sustained_active", "smsp__inst_executed.sum",
    "sm__cycles_elapsed.max", "lts__t_sector_hit_rate.pct",
    "smsp__average_warps_issue_stalled_math_pipe_throttle_per_issue_active.ratio",
    "smsp__average_warps_issue_stalled_wait_per_issue_active.ratio",
    "smsp__average_warps_issue_stalled_barrier_per_issue_active.ratio",
    "smsp__average_warps_issue_stalled_short_scoreboard_per_issue_active.ratio",
    "smsp__average_warps_issue_stalled_long_scoreboard_per_issue_active.ratio",
    "smsp__average_warps_issue_stalled_mio_throttle_per_issue_active.ratio",
]


def source_digest() -> str:
    """SHA-256 over the kernel sources (the .cuh files under csrc/, where every kernel and its
    launch configuration live; the .cu files only select and launch), in name order."""
    h = hashlib.sha256()
    for path in sorted(glob.glob(os.path.join(PKG, "csrc", "*.cuh"))):
        h.update(os.path.basename(path).encode())
        with open(path, "rb") as f:
            h.update(f.read())
    return h.hexdigest()[:16]


def read_report(path: str, kernel: str):
    out = subprocess.run(["ncu", "-i", path, "--page", "raw", "--csv"], capture_output=True,
                         text=True, check=True).stdout
    rows = list(csv.reader(out.splitlines()))
    hdr, units, body = rows[0], rows[1], rows[2:]
    name_col = hdr.index("Kernel Name")
    body = [r for r in body if re.search(kernel, r[name_col])]
    if not body:
        raise SystemExit(f"no launch of a kernel matching {kernel!r} in {path}")
    return hdr, units, body, body[0][name_col]


def to_bytes(value: str, unit: str) -> float:
    scale = {"byte": 1.0, "Kbyte": 1e3, "Mbyte": 1e6, "Gbyte": 1e9}[unit]
    return float(value.replace(",", "")) * scale


def main(argv=None):
    ap = argparse.ArgumentParser()
    ap.add_argument("report")
    ap.add_argument("--kernel", required=True)
    ap.add_argument("--workload", default=None, help="key in profiles/dram_traffic.json")
    ap.add_argument("--elements", type=int, default=0, help="elements one captured launch processed")
    ap.add_argument("--out", default=None)
    ap.add_argument("--command", default="")
    args = ap.parse_args(argv)
    hdr, units, body, name = read_report(args.report, args.kernel)
    lines = [f"# `{name}` -- ncu summary", ""]
    if args.command:
        lines += ["Command (run after the same command had exited 0 without ncu):", "",
                  "    " + args.command, ""]
    lines += [f"{len(body)} launch(es) captured; values are given launch by launch.", "",
              "| metric | unit | value |", "|---|---|---|"]
    for m in METRICS:
        if m in hdr:
            i = hdr.index(m)
            lines.append(f"| `{m}` | {units[i]} | {' / '.join(r[i] for r in body)} |")
    ir, iw = hdr.index("dram__bytes_read.sum"), hdr.index("dram__bytes_write.sum")
    traffic = sum(to_bytes(r[ir], units[ir]) + to_bytes(r[iw], units[iw]) for r in body) / len(body)
    lines += ["", f"DRAM traffic per launch (read + write, mean over the launches): {traffic:.0f} bytes"]
    if args.elements:
        lines.append(f"= {traffic / args.elements:.1f} bytes per element ({args.elements} elements per launch)")
    text = "\n".join(lines) + "\n"
    if args.out:
        with open(args.out, "w") as f:
            f.write(text)
    else:
        sys.stdout.write(text)
    if args.workload:
        if not args.elements:
            raise SystemExit("--workload needs --elements")
        data = {}
        if os.path.exists(TRAFFIC_JSON):
            with open(TRAFFIC_JSON) as f:
                data = json.load(f)
        data[args.workload] = {"bytes_per_element": traffic / args.elements, "kernel": name,
                               "captured_elements": args.elements,
                               "source_digest": source_digest()}
        with open(TRAFFIC_JSON, "w") as f:
            json.dump(data, f, indent=1, sort_keys=True)
            f.write("\n")


if __name__ == "__main__":
    main()
