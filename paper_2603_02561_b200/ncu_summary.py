"""Turns the raw-page CSV of an ncu report into a short text summary and records the kernel's
DRAM traffic per launch.

    ncu -i prof.ncu-rep --page raw --csv > prof.csv
    python -m paper_2603_02561_b200.ncu_summary prof.csv --kernel eig --workload c3 \\
        --source paper_2603_02561_b200/csrc/eig_tridiag.cu --command "<the command that was profiled>" \\
        --out profiles/eig_tridiag_c3.md [--traffic profiles/traffic.json]
    python -m paper_2603_02561_b200.ncu_summary launch-list launches.csv --command "<...>" --out profiles/launches_bench_c3.md

The traffic file maps "<workload>/<kernel>" to the bytes per launch (dram__bytes_read.sum +
dram__bytes_write.sum, averaged over the captured launches) and to a hash of the kernel's
source file at capture time; the benchmark reports the figure only while the hash still
matches, so a number taken before the kernel changed is never shown as current.
"""
from __future__ import annotations

import argparse
import csv
import hashlib
import json
import os

KEEP = [
    "gpu__time_duration.sum", "launch__registers_per_thread", "launch__grid_size", "launch__block_size",
    "launch__shared_mem_per_block_dynamic", "launch__occupancy_limit_registers", "launch__occupancy_limit_shared_mem",
    "dram__bytes_read.sum", "dram__bytes_write.sum", "gpu__dram_throughput.avg.pct_of_peak_sustained_elapsed",
    "lts__t_bytes.sum", "sm__throughput.avg.pct_of_peak_sustained_elapsed",
    "sm__pipe_tensor_cycles_active.avg.pct_of_peak_sustained_active", "sm__warps_active.avg.pct_of_peak_sustained_active",
    "smsp__inst_executed.sum", "smsp__issue_active.avg.pct", "sm__inst_executed_pipe_xu.sum",
    "smsp__average_warps_issue_stalled_long_scoreboard_per_issue_active.ratio",
    "smsp__average_warps_issue_stalled_short_scoreboard_per_issue_active.ratio",
    "smsp__average_warps_issue_stalled_barrier_per_issue_active.ratio",
    "smsp__average_warps_issue_stalled_wait_per_issue_active.ratio",
    "smsp__average_warps_issue_stalled_no_instruction_per_issue_active.ratio",
    "smsp__average_warps_issue_stalled_branch_resolving_per_issue_active.ratio",
    "l1tex__data_bank_conflicts_pipe_lsu_mem_shared.sum", "l1tex__data_pipe_lsu_wavefronts_mem_shared.sum",
]


def source_hash(path: str) -> str:
    with open(path, "rb") as f:
        return hashlib.sha1(f.read()).hexdigest()[:16]


def read_raw(path: str):
    rows = list(csv.reader(open(path)))
    hdr = rows[0]
    units = rows[1]
    launches = rows[2:]
    return hdr, units, launches


def launch_list(path: str, out: str, command: str):
    """Per kernel: launches, total device time and share, from the CSV log of
    `ncu --metrics gpu__time_duration.sum --csv --log-file <path>`."""
    import collections
    import re
    with open(path) as f:
        lines = [ln for ln in f if ln.startswith('"')]
    agg = collections.OrderedDict()
    for r in csv.DictReader(lines):
        if r["Metric Name"] != "gpu__time_duration.sum":
            continue
        short = re.sub(r"^void ", "", re.sub(r"\(.*", "", r["Kernel Name"]))[:90]
        ns = float(r["Metric Value"].replace(",", "")) * {"ns": 1, "us": 1e3, "ms": 1e6}.get(r["Metric Unit"], 1)
        a = agg.setdefault((short, r["Grid Size"], r["Block Size"]), [0, 0.0])
        a[0] += 1
        a[1] += ns
    tot = sum(v[1] for v in agg.values())
    rows = [f"# ncu launch list", "", f"Command: `{command}`", "",
            "Per-launch times under ncu are cold-cache and serialised: compare the shares, not the absolutes.", "",
            "| kernel | grid | block | launches | total us | avg us | share |", "|---|---|---|---|---|---|---|"]
    for (k, g, b), (n, t) in sorted(agg.items(), key=lambda kv: -kv[1][1]):
        rows.append(f"| {k} | {g} | {b} | {n} | {t / 1e3:.1f} | {t / 1e3 / n:.2f} | {100 * t / tot:.1f}% |")
    rows += ["", f"total {tot / 1e3:.1f} us over {sum(v[0] for v in agg.values())} launches", ""]
    open(out, "w").write("\n".join(rows))
    print(f"wrote {out}")


def main():
    import sys
    if len(sys.argv) > 1 and sys.argv[1] == "launch-list":
        ap = argparse.ArgumentParser()
        ap.add_argument("mode")
        ap.add_argument("csv")
        ap.add_argument("--command", required=True)
        ap.add_argument("--out", required=True)
        a = ap.parse_args()
        launch_list(a.csv, a.out, a.command)
        return
    ap = argparse.ArgumentParser()
    ap.add_argument("csv")
    ap.add_argument("--kernel", required=True, help="short name used by the benchmark (gram, eig, attn_apply, ...)")
    ap.add_argument("--workload", required=True)
    ap.add_argument("--source", required=True, help="the kernel's source file (hashed)")
    ap.add_argument("--command", required=True)
    ap.add_argument("--out", required=True)
    ap.add_argument("--traffic", default=None)
    ap.add_argument("--note", default="")
    args = ap.parse_args()
    hdr, units, launches = read_raw(args.csv)
    col = {h: i for i, h in enumerate(hdr)}
    name_col = col.get("Kernel Name")
    lines = [f"# ncu summary: {args.kernel} on {args.workload}", "",
             f"Command: `{args.command}`", "",
             f"Kernel source: `{args.source}` (sha1 {source_hash(args.source)}); {len(launches)} launch(es) captured"
             + (f": {launches[0][name_col][:100]}" if name_col is not None and launches else ""), ""]
    if args.note:
        lines += [args.note, ""]
    lines += ["| metric | unit | " + " | ".join(f"launch {i + 1}" for i in range(len(launches))) + " |",
              "|---|---|" + "---|" * len(launches)]

    def num(x):
        try:
            return float(x.replace(",", ""))
        except ValueError:
            return None
    for m in KEEP:
        if m in col:
            vals = [r[col[m]] for r in launches]
            lines.append(f"| {m} | {units[col[m]]} | " + " | ".join(vals) + " |")
    dram = []
    for r in launches:
        rd, wr = num(r[col["dram__bytes_read.sum"]]), num(r[col["dram__bytes_write.sum"]])
        scale = {"byte": 1, "Kbyte": 1e3, "Mbyte": 1e6, "Gbyte": 1e9}
        ur, uw = units[col["dram__bytes_read.sum"]], units[col["dram__bytes_write.sum"]]
        dram.append(rd * scale.get(ur, 1) + wr * scale.get(uw, 1))
    per_launch = sum(dram) / max(1, len(dram))
    lines += ["", f"DRAM traffic per launch (read + write, mean of the captured launches): {per_launch / 1e6:.3f} MB", ""]
    os.makedirs(os.path.dirname(args.out) or ".", exist_ok=True)
    open(args.out, "w").write("\n".join(lines))
    if args.traffic:
        data = json.load(open(args.traffic)) if os.path.exists(args.traffic) else {}
        data[f"{args.workload}/{args.kernel}"] = {"dram_bytes_per_launch": per_launch, "source": args.source,
                                                   "source_sha1": source_hash(args.source), "summary": args.out}
        json.dump(data, open(args.traffic, "w"), indent=1, sort_keys=True)
    print(f"wrote {args.out}: {per_launch / 1e6:.3f} MB per launch")


if __name__ == "__main__":
    main()
