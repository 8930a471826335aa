"""Turns an Nsight Compute report into the short text summary kept under ``profiles/`` and records the DRAM traffic of
the attention kernel in ``profiles/traffic.json``, which ``bench.py`` reads for ``roofline.traffic``.

    python -m paper_2506_19830_b200.ncu_summary report.ncu-rep --out profiles/attention_config3.txt \
        --title "lr_verify_attention on config 3" --command "ncu --set full ... python bench.py ..." \
        [more reports, more --command lines] \
        [--traffic-workload config3_long_context --traffic-kernel attn_tc_kernel]

    python -m paper_2506_19830_b200.ncu_summary launches.csv --launch-list --out profiles/launch_list.txt ...

The first form needs ``ncu`` on the PATH (it only reads the report: no GPU).  A traffic record carries the SHA-256 of
the kernel's source file as it is when the summary is written; ``bench.py`` reports the traffic only while the
source still has that hash.
"""
from __future__ import annotations

import argparse
import csv
import hashlib
import io
import json
import os
import subprocess
import sys
from collections import OrderedDict

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
KERNEL_SOURCES = {"attn_tc_kernel": "attn_tc.cu", "attn_pair_kernel": "attn_pair.cu"}

KEYS = [
    "gpu__time_duration.sum", "dram__bytes_read.sum", "dram__bytes_write.sum",
    "gpu__dram_throughput.avg.pct_of_peak_sustained_elapsed",
    "sm__pipe_tensor_cycles_active.avg.pct_of_peak_sustained_active",
    "sm__inst_executed_pipe_xu.avg.pct_of_peak_sustained_active",
    "smsp__issue_active.avg.pct_of_peak_sustained_active", "sm__warps_active.avg.pct_of_peak_sustained_active",
    "launch__registers_per_thread", "launch__grid_size", "launch__block_size", "launch__cluster_size",
    "smsp__inst_executed.sum", "lts__t_sector_hit_rate.pct",
    "smsp__average_warps_issue_stalled_long_scoreboard_per_issue_active.ratio",
    "smsp__average_warps_issue_stalled_wait_per_issue_active.ratio",
    "smsp__average_warps_issue_stalled_math_pipe_throttle_per_issue_active.ratio",
    "smsp__average_warps_issue_stalled_barrier_per_issue_active.ratio",
    "smsp__average_warps_issue_stalled_short_scoreboard_per_issue_active.ratio",
    "smsp__average_warps_issue_stalled_no_instruction_per_issue_active.ratio",
]
TO_BYTES = {"byte": 1, "Kbyte": 1e3, "Mbyte": 1e6, "Gbyte": 1e9}


def read_report(path: str):
    """Rows of the report's raw page: a list of (kernel name, {metric: (value, unit)})."""
    out = subprocess.run(["ncu", "-i", path, "--page", "raw", "--csv"], capture_output=True, text=True, check=True).stdout
    rows = list(csv.reader(io.StringIO(out)))
    header, units = rows[0], rows[1]
    launches = []
    for r in rows[2:]:
        d = OrderedDict((k, (v, u)) for k, v, u in zip(header, r, units))
        launches.append((d.get("Kernel Name", ("?", ""))[0], d))
    return launches


def summarise(launches) -> str:
    lines = []
    for name, d in launches:
        lines.append(f"launch: {name[:110]}")
        for k in KEYS:
            if k in d:
                v, u = d[k]
                lines.append(f"  {k:<86} {v} {u}")
        lines.append("")
    return "\n".join(lines)


def launch_list(path: str) -> str:
    """Per kernel: launches, total time, share -- from the CSV log of an ncu run with gpu__time_duration.sum alone."""
    text = open(path).read()
    start = text.find('"ID"')
    rows = list(csv.DictReader(io.StringIO(text[start:])))
    per = OrderedDict()
    for r in rows:
        if r.get("Metric Name") != "gpu__time_duration.sum":
            continue
        v = float(r["Metric Value"].replace(",", ""))
        unit = r.get("Metric Unit", "ns")
        ns = v * {"ns": 1.0, "us": 1e3, "usecond": 1e3, "ms": 1e6, "msecond": 1e6, "nsecond": 1.0}.get(unit, 1.0)
        name = r["Kernel Name"].split("(")[0]
        n, t = per.get(name, (0, 0.0))
        per[name] = (n + 1, t + ns)
    total = sum(t for _, t in per.values()) or 1.0
    lines = [f"{'kernel':<60} {'launches':>8} {'total us':>10} {'share':>7}"]
    for name, (n, t) in sorted(per.items(), key=lambda kv: -kv[1][1]):
        lines.append(f"{name[-60:]:<60} {n:>8} {t / 1e3:>10.1f} {t / total:>7.1%}")
    return "\n".join(lines) + "\n"


def record_traffic(launches, workload: str, kernel: str) -> None:
    for name, d in launches:
        if kernel in name:
            rd = float(d["dram__bytes_read.sum"][0].replace(",", "")) * TO_BYTES[d["dram__bytes_read.sum"][1]]
            wr = float(d["dram__bytes_write.sum"][0].replace(",", "")) * TO_BYTES[d["dram__bytes_write.sum"][1]]
            src = os.path.join(ROOT, "paper_2506_19830_b200", "csrc", KERNEL_SOURCES[kernel])
            path = os.path.join(ROOT, "profiles", "traffic.json")
            table = json.load(open(path)) if os.path.exists(path) else {}
            table.setdefault(workload, {})[kernel] = {
                "dram_bytes_read": int(rd), "dram_bytes_write": int(wr),
                "source_sha256": hashlib.sha256(open(src, "rb").read()).hexdigest(), "source": KERNEL_SOURCES[kernel]}
            json.dump(table, open(path, "w"), indent=1, sort_keys=True)
            return
    raise SystemExit(f"no launch of {kernel} in the report")


def main() -> int:
    ap = argparse.ArgumentParser()
    ap.add_argument("report", nargs="+", help="one or more reports (their launches are listed one after another)")
    ap.add_argument("--out", required=True)
    ap.add_argument("--title", default="")
    ap.add_argument("--command", action="append", default=[], help="the full command that produced a report (repeatable)")
    ap.add_argument("--note", action="append", default=[])
    ap.add_argument("--launch-list", action="store_true")
    ap.add_argument("--traffic-workload", default="")
    ap.add_argument("--traffic-kernel", default="attn_tc_kernel")
    a = ap.parse_args()
    head = [f"# {a.title}", "# command (B200, one GPU; each preceded by the same command without ncu exiting 0):"]
    head += [f"#   {c}" for c in a.command]
    head += [f"# {n}" for n in a.note]
    if a.launch_list:
        body = launch_list(a.report[0])
    else:
        launches = [l for r in a.report for l in read_report(r)]
        body = summarise(launches)
        if a.traffic_workload:
            record_traffic(launches, a.traffic_workload, a.traffic_kernel)
    with open(a.out, "w") as f:
        f.write("\n".join(head) + "\n\n" + body)
    return 0


if __name__ == "__main__":
    sys.exit(main())
