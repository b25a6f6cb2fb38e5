"""Turns an Nsight Compute report into the short text tables kept under profiles/.

    python -m paper_2503_08154_b200.ncu_summary table  <report.ncu-rep> [more reports] [--title T] [--command C]
    python -m paper_2503_08154_b200.ncu_summary launches <launches.csv> [--title T] [--command C]
    python -m paper_2503_08154_b200.ncu_summary traffic <report.ncu-rep> [more reports] --workload NAME [--skip-first N]

`table` prints one column per captured launch with the counters the roofline discussion uses
(duration, DRAM bytes and throughput, issue and pipe utilisation, stalls, registers).
`launches` reads the CSV log of a `--metrics gpu__time_duration.sum` run and prints launches,
total time and share per kernel.  `traffic` prints the JSON that profiles/traffic.json
holds: DRAM bytes per launch per kernel (mean over the captured launches), stamped with a
digest of the kernel sources so that bench.py can tell when it is stale.

The report is read with `ncu -i <report> --page raw --csv`; nothing here needs a GPU.
"""
from __future__ import annotations

import argparse
import csv
import hashlib
import io
import json
import os
import re
import subprocess
import sys
from collections import OrderedDict

HERE = os.path.dirname(os.path.abspath(__file__))

# (label, metric name as ncu prints it, scale)
ROWS = [
    ("gpu__time_duration.sum [us]", "gpu__time_duration.sum", None),
    ("dram__bytes_read.sum [MB]", "dram__bytes_read.sum", None),
    ("dram__bytes_write.sum [MB]", "dram__bytes_write.sum", None),
    ("gpu__dram_throughput % of peak", "gpu__dram_throughput.avg.pct_of_peak_sustained_elapsed", None),
    ("dram__cycles_active % of peak", "dram__cycles_active.avg.pct_of_peak_sustained_elapsed", None),
    ("sm__throughput % of peak", "sm__throughput.avg.pct_of_peak_sustained_elapsed", None),
    ("smsp__issue_active %", "smsp__issue_active.avg.pct_of_peak_sustained_active", None),
    ("smsp__inst_executed.sum", "smsp__inst_executed.sum", None),
    ("sm__warps_active % of peak", "sm__warps_active.avg.pct_of_peak_sustained_active", None),
    ("pipe xu %", "sm__inst_executed_pipe_xu.avg.pct_of_peak_sustained_active", None),
    ("pipe alu %", "sm__pipe_alu_cycles_active.avg.pct_of_peak_sustained_active", None),
    ("pipe fma %", "sm__pipe_fma_cycles_active.avg.pct_of_peak_sustained_active", None),
    ("shared bank conflicts", "l1tex__data_bank_conflicts_pipe_lsu_mem_shared.sum", None),
    ("registers / thread", "launch__registers_per_thread", None),
    ("grid", "launch__grid_size", None),
    ("block", "launch__block_size", None),
    ("stall long_scoreboard / issue", "smsp__average_warps_issue_stalled_long_scoreboard_per_issue_active.ratio", None),
    ("stall short_scoreboard / issue", "smsp__average_warps_issue_stalled_short_scoreboard_per_issue_active.ratio", None),
    ("stall wait / issue", "smsp__average_warps_issue_stalled_wait_per_issue_active.ratio", None),
    ("stall not_selected / issue", "smsp__average_warps_issue_stalled_not_selected_per_issue_active.ratio", None),
    ("stall math_pipe_throttle / issue", "smsp__average_warps_issue_stalled_math_pipe_throttle_per_issue_active.ratio", None),
    ("stall barrier / issue", "smsp__average_warps_issue_stalled_barrier_per_issue_active.ratio", None),
    ("stall mio_throttle / issue", "smsp__average_warps_issue_stalled_mio_throttle_per_issue_active.ratio", None),
]
UNIT_TO_BYTES = {"byte": 1.0, "Kbyte": 1e3, "Mbyte": 1e6, "Gbyte": 1e9}
UNIT_TO_US = {"ns": 1e-3, "us": 1.0, "ms": 1e3, "s": 1e6, "nsecond": 1e-3, "usecond": 1.0, "msecond": 1e3, "second": 1e6}


def read_raw(report: str):
    """Returns (list of launches); each launch is {"name": ..., metric: (value, unit)}."""
    out = subprocess.run(["ncu", "-i", report, "--page", "raw", "--csv", "--print-kernel-base", "demangled"],
                         capture_output=True, text=True, check=True).stdout
    rows = list(csv.reader(io.StringIO(out)))
    header, units = rows[0], rows[1]
    launches = []
    for r in rows[2:]:
        if len(r) != len(header):
            continue
        d = {"name": r[header.index("Kernel Name")]}
        for h, u, v in zip(header, units, r):
            try:
                d[h] = (float(v.replace(",", "")), u)
            except ValueError:
                pass
        launches.append(d)
    return launches


def short_name(name: str) -> str:
    m = re.search(r"tile_kernel<(?:.*?::)?(\w+<[^>]*>)", name)
    s = m.group(1) if m else name.split("(")[0]
    return re.sub(r"\(int\)", "", s)


def fmt(metric, d):
    if metric not in d:
        return "n/a"
    v, u = d[metric]
    if metric.startswith("dram__bytes"):
        return "%.3f" % (v * UNIT_TO_BYTES.get(u, 1.0) / 1e6)
    if metric == "gpu__time_duration.sum":
        return "%.3f" % (v * UNIT_TO_US.get(u, 1.0))
    return ("%.0f" % v) if abs(v) >= 1000 else ("%.3f" % v)


def cmd_table(args):
    launches = []
    for rep in [args.report] + list(args.more):
        launches += read_raw(rep)
    if args.title:
        print(args.title)
    if args.command:
        print("command: " + args.command)
    print("read with: ncu -i <report> --page raw --csv --print-kernel-base demangled  (python -m paper_2503_08154_b200.ncu_summary table <report>)")
    print()
    names = ["%d:%s" % (i, short_name(d["name"])[:26]) for i, d in enumerate(launches)]
    w = max(28, max(len(n) for n in names) + 2)
    print("%-34s" % "metric" + "".join("%*s" % (w, n) for n in names))
    for label, metric, _ in ROWS:
        if not any(metric in d for d in launches):
            continue
        print("%-34s" % label + "".join("%*s" % (w, fmt(metric, d)) for d in launches))
    print()
    print("DRAM traffic per launch (read + write), MB: " +
          ", ".join("%s %.1f" % (n, (d.get("dram__bytes_read.sum", (0, "byte"))[0] * UNIT_TO_BYTES.get(d.get("dram__bytes_read.sum", (0, "byte"))[1], 1) +
                                     d.get("dram__bytes_write.sum", (0, "byte"))[0] * UNIT_TO_BYTES.get(d.get("dram__bytes_write.sum", (0, "byte"))[1], 1)) / 1e6)
                    for n, d in zip(names, launches)))


def cmd_launches(args):
    text = open(args.report).read()
    start = text.index('"ID"')
    rows = list(csv.DictReader(io.StringIO(text[start:])))
    per = OrderedDict()
    for r in rows:
        if r.get("Metric Name") != "gpu__time_duration.sum":
            continue
        v = float(r["Metric Value"].replace(",", "")) * UNIT_TO_US.get(r["Metric Unit"], 1.0)
        per.setdefault(short_name(r["Kernel Name"]), []).append(v)
    total = sum(sum(v) for v in per.values())
    if args.title:
        print(args.title)
    if args.command:
        print("command: " + args.command)
    print("(per-launch times under ncu are cold-cache and serialised; compare SHARES with bench.py per_kernel.share_of_step)")
    print()
    print("%-44s %9s %14s %12s %7s" % ("kernel", "launches", "total us", "avg us", "share"))
    for k, v in per.items():
        print("%-44s %9d %14.1f %12.2f %6.1f%%" % (k[:44], len(v), sum(v), sum(v) / len(v), 100 * sum(v) / total))


def kernel_source_digest():
    h = hashlib.sha256()
    csrc = os.path.join(HERE, "csrc")
    for name in sorted(os.listdir(csrc)):
        h.update(open(os.path.join(csrc, name), "rb").read())
    return h.hexdigest()[:16]


KIND = (("SoftmaxFwd", "softmax_fwd"), ("SoftmaxBwd", "softmax_bwd"), ("ActFwd", "gelu_fwd"), ("ActBwd", "gelu_bwd"))


def cmd_traffic(args):
    launches = []
    for rep in [args.report] + list(args.more):
        launches += read_raw(rep)[args.skip_first:]
    per = {}
    for d in launches:
        kind = next((k for pat, k in KIND if pat in d["name"]), None)
        if kind is None or "dram__bytes_read.sum" not in d:
            continue
        rd = d["dram__bytes_read.sum"][0] * UNIT_TO_BYTES.get(d["dram__bytes_read.sum"][1], 1.0)
        wr = d["dram__bytes_write.sum"][0] * UNIT_TO_BYTES.get(d["dram__bytes_write.sum"][1], 1.0)
        per.setdefault(kind, []).append((rd, wr))
    digest = kernel_source_digest()
    out = {args.workload: {k: {"dram_bytes_per_launch": int(sum(r + w for r, w in v) / len(v)),
                               "read": int(sum(r for r, _ in v) / len(v)), "write": int(sum(w for _, w in v) / len(v)),
                               "launches": len(v), "source_digest": digest, "capture": args.note}
                           for k, v in per.items()}}
    print(json.dumps(out, indent=1))


def main():
    ap = argparse.ArgumentParser()
    sub = ap.add_subparsers(dest="cmd", required=True)
    for name in ("table", "launches", "traffic"):
        p = sub.add_parser(name)
        p.add_argument("report")
        p.add_argument("more", nargs="*", help="further reports, appended (table and traffic)")
        p.add_argument("--title", default="")
        p.add_argument("--command", default="")
        if name == "traffic":
            p.add_argument("--workload", required=True)
            p.add_argument("--skip-first", type=int, default=0)
            p.add_argument("--note", default="")
    args = ap.parse_args()
    {"table": cmd_table, "launches": cmd_launches, "traffic": cmd_traffic}[args.cmd](args)


if __name__ == "__main__":
    sys.exit(main())
