"""Turns Nsight Compute output into the short records kept under profiles/.

  python -m paper_2507_19131_b200.ncu_summary launches out/launches.csv
      per kernel: launches, total time, share (from `ncu --metrics gpu__time_duration.sum --csv --log-file ...`)

  python -m paper_2507_19131_b200.ncu_summary traffic out/gemm_traffic.ncu-rep --workload cfg3-swin_t-800x1333 \
         --fc1-outputs 130351104
      DRAM bytes of the GEMM launches of ONE forward (the report must hold exactly the GEMM launches of one forward:
      `ncu --metrics dram__bytes_read.sum,dram__bytes_write.sum,smsp__inst_executed.sum -k regex:k_gemm_tc -c <n>`),
      written to profiles/ncu_dram_traffic.json together with a digest of the kernel sources; bench.py reports the
      figures only while the digest still matches the sources it runs.

  python -m paper_2507_19131_b200.ncu_summary metrics some.ncu-rep [metric ...]
      one line per metric, one column per captured launch (for the .md summaries)
"""
from __future__ import annotations

import argparse
import collections
import csv
import hashlib
import json
import os
import re
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(HERE)
TRAFFIC_JSON = os.path.join(ROOT, "profiles", "ncu_dram_traffic.json")

# template argument of k_gemm_tc -> the category name the library's profiling hooks use
GEMM_MODE_CATEGORY = {0: "gemm_qkv", 1: "gemm_proj", 2: "gemm_fc1_gelu", 3: "gemm_fc2_scatter", 4: "gemm_merge"}

DEFAULT_METRICS = [
    "gpu__time_duration.sum", "dram__bytes_read.sum", "dram__bytes_write.sum",
    "gpu__dram_throughput.avg.pct_of_peak_sustained_elapsed",
    "sm__pipe_tensor_cycles_active.avg.pct_of_peak_sustained_active",
    "sm__warps_active.avg.pct_of_peak_sustained_active", "launch__registers_per_thread",
    "smsp__inst_executed.sum", "smsp__issue_active.avg.pct_of_peak_sustained_active",
    "sm__inst_executed_pipe_fma.sum.pct_of_peak_sustained_active",
    "sm__inst_executed_pipe_alu.sum.pct_of_peak_sustained_active",
    "sm__inst_executed_pipe_lsu.sum.pct_of_peak_sustained_active",
    "l1tex__data_bank_conflicts_pipe_lsu_mem_shared.sum",
    "smsp__average_warps_issue_stalled_long_scoreboard_per_issue_active.ratio",
    "smsp__average_warps_issue_stalled_short_scoreboard_per_issue_active.ratio",
    "smsp__average_warps_issue_stalled_barrier_per_issue_active.ratio",
    "smsp__average_warps_issue_stalled_math_pipe_throttle_per_issue_active.ratio",
    "smsp__average_warps_issue_stalled_not_selected_per_issue_active.ratio",
]


# the sources that hold the device code of the GEMM kernel whose DRAM traffic is recorded
GEMM_KERNEL_SOURCES = ("common.cuh", "gemm_epilogue.cuh", "gemm_tc.cu", "kernels.h")


def kernel_source_digest() -> str:
    """sha256 (first 16 hex digits) over the sources of the GEMM kernel."""
    h = hashlib.sha256()
    csrc = os.path.join(HERE, "csrc")
    for f in GEMM_KERNEL_SOURCES:
        h.update(f.encode())
        h.update(open(os.path.join(csrc, f), "rb").read())
    return h.hexdigest()[:16]


def raw_rows(report: str):
    """(header, units, rows) of `ncu -i report --page raw --csv`; a .csv file is read as that output."""
    if report.endswith(".csv"):
        text = open(report).read()
    else:
        text = subprocess.run(["ncu", "-i", report, "--page", "raw", "--csv"], capture_output=True, text=True, check=True).stdout
    rows = list(csv.reader([l for l in text.splitlines() if l.startswith('"')]))
    return rows[0], rows[1], rows[2:]


def to_bytes(value: str, unit: str) -> float:
    scale = {"byte": 1.0, "Kbyte": 1e3, "Mbyte": 1e6, "Gbyte": 1e9}
    return float(value.replace(",", "")) * scale.get(unit, 1.0)


def cmd_launches(args):
    lines = [l for l in open(args.csv) if l.startswith('"')]
    agg = collections.OrderedDict()
    for r in csv.DictReader(lines):
        name = re.sub(r"\(.*", "", r["Kernel Name"]).replace("mixaq::", "").replace("(anonymous namespace)::", "")
        a = agg.setdefault(name, [0, 0.0])
        a[0] += 1
        a[1] += float(r["Metric Value"].replace(",", ""))
    total = sum(a[1] for a in agg.values())
    print(f"{'kernel':60s} {'launches':>8s} {'total_us':>10s} {'share':>7s}")
    for name, (n, t) in sorted(agg.items(), key=lambda kv: -kv[1][1]):
        print(f"{name[:60]:60s} {n:8d} {t / 1e3:10.1f} {t / total:7.3f}")


def cmd_metrics(args):
    hdr, units, rows = raw_rows(args.report)
    idx = {h: i for i, h in enumerate(hdr)}
    print("metric | " + " | ".join(r[idx["Kernel Name"]][:34] + " " + r[idx["Grid Size"]] for r in rows))
    for k in (args.metric or DEFAULT_METRICS):
        if k in idx:
            short = k.replace("smsp__average_warps_issue_stalled_", "stall_").replace("_per_issue_active.ratio", "")
            print(short, units[idx[k]], "|", " | ".join(r[idx[k]][:12] for r in rows))


def cmd_traffic(args):
    hdr, units, rows = raw_rows(args.report)
    idx = {h: i for i, h in enumerate(hdr)}
    per_cat = collections.OrderedDict((c, 0.0) for c in GEMM_MODE_CATEGORY.values())
    launches = collections.Counter()
    fc1_inst = 0.0
    for r in rows:
        m = re.search(r"k_gemm_tc<\(?(?:int\))?(\d)", r[idx["Kernel Name"]])
        if not m:
            continue
        cat = GEMM_MODE_CATEGORY[int(m.group(1))]
        b = sum(to_bytes(r[idx[k]], units[idx[k]]) for k in ("dram__bytes_read.sum", "dram__bytes_write.sum"))
        per_cat[cat] += b
        launches[cat] += 1
        if cat == "gemm_fc1_gelu" and "smsp__inst_executed.sum" in idx:
            fc1_inst += float(r[idx["smsp__inst_executed.sum"]].replace(",", ""))
    rec = {"kernel_source_digest": kernel_source_digest(), "bytes_per_step": per_cat, "launches_per_step": dict(launches),
           "source": os.path.basename(args.report),
           "how": "dram__bytes_read.sum + dram__bytes_write.sum summed over the GEMM launches of one forward (one ncu capture)"}
    if args.command:
        rec["command"] = args.command
    if args.fc1_outputs and fc1_inst:
        rec["fc1_warp_inst_per_32_outputs"] = round(fc1_inst / (args.fc1_outputs / 32.0), 2)
    data = {}
    if os.path.exists(TRAFFIC_JSON):
        data = json.load(open(TRAFFIC_JSON))
    data[args.workload] = rec
    json.dump(data, open(TRAFFIC_JSON, "w"), indent=1)
    print(json.dumps(rec, indent=1))


def main():
    ap = argparse.ArgumentParser()
    sub = ap.add_subparsers(dest="cmd", required=True)
    a = sub.add_parser("launches"); a.add_argument("csv"); a.set_defaults(fn=cmd_launches)
    a = sub.add_parser("metrics"); a.add_argument("report"); a.add_argument("metric", nargs="*"); a.set_defaults(fn=cmd_metrics)
    a = sub.add_parser("traffic"); a.add_argument("report"); a.add_argument("--workload", required=True)
    a.add_argument("--fc1-outputs", type=float, default=0.0, help="fc1 outputs (rows x hidden) of one forward")
    a.add_argument("--command", default="", help="the full ncu command that produced the report (kept in the record)")
    a.set_defaults(fn=cmd_traffic)
    args = ap.parse_args()
    args.fn(args)


if __name__ == "__main__":
    sys.exit(main())
