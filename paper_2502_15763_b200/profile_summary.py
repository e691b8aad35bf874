"""Turns one Nsight Compute report of a `bench.py` run into the small counter file that `bench.py`
reads for its `traffic` figures (DRAM bytes and warp instructions per unit of work and kernel).

    python -m paper_2502_15763_b200.profile_summary REPORT.ncu-rep BENCH_LINE.json -o profiles/NAME.json \
        --command "the ncu command that made the report"

REPORT is read with `ncu -i REPORT --page raw --csv` (no GPU needed).  BENCH_LINE is the JSON line
that the same `bench.py` command printed when it ran without the profiler: it gives the units
one launch processed (requests, simulated iterations, executed local-search rounds).  The file
records the hash of the library sources, and `bench.py` ignores it once the sources have changed.
"""
from __future__ import annotations

import argparse
import csv
import io
import json
import re
import subprocess

from . import _build

# unit of work of every kernel: its DRAM traffic and instruction count grow in proportion to it
UNIT = {"k_estimate_sort": "request", "k_lpt": "request", "k_ls_lists": "request", "k_multifit": "request",
        "k_queue_build": "request", "k_simulate": "request", "k_simulate_steal": "request",
        "k_local_search": "round", "k_trace_fill": "iteration"}
COUNTERS = {
    "time_us": "gpu__time_duration.sum",
    "dram_read": "dram__bytes_read.sum",
    "dram_write": "dram__bytes_write.sum",
    "warp_inst": "smsp__inst_executed.sum",
    "issue_active_pct": "smsp__issue_active.avg.pct_of_peak_sustained_active",
    "warps_active_pct": "sm__warps_active.avg.pct_of_peak_sustained_active",
    "threads_per_inst": "smsp__thread_inst_executed_per_inst_executed.ratio",
    "dram_throughput_pct": "gpu__dram_throughput.avg.pct_of_peak_sustained_elapsed",
    "registers": "launch__registers_per_thread",
}
SCALE = {"byte": 1.0, "Kbyte": 1e3, "Mbyte": 1e6, "Gbyte": 1e9, "us": 1.0, "ms": 1e3, "ns": 1e-3, "s": 1e6,
         "usecond": 1.0, "msecond": 1e3, "nsecond": 1e-3, "second": 1e6}


def short_name(full: str) -> str:
    """hos::k_simulate<hos::NarrowEntry>(...) -> k_simulate; the radix fallbacks and the wide
    instantiations (which return at once on ordinary inputs) keep a suffix."""
    m = re.search(r"(k_[a-z_]+)(<[^>(]*>)?", full)
    name = m.group(1) if m else full
    args = m.group(2) or "" if m else ""
    if name in ("k_estimate_sort", "k_queue_build") and ("<0>" in args or "false" in args):
        name += "_radix"
    if "WideEntry" in args:
        name += "_wide"
    return name


def read_report(path: str):
    text = subprocess.run(["ncu", "-i", path, "--page", "raw", "--csv"], check=True, capture_output=True,
                          text=True).stdout
    rows = list(csv.reader(io.StringIO(text)))
    hdr, units = rows[0], rows[1]
    col = {h: i for i, h in enumerate(hdr)}
    out = []
    for r in rows[2:]:
        rec = {"kernel": short_name(r[col["Kernel Name"]])}
        for key, metric in COUNTERS.items():
            if metric not in col:
                continue
            try:
                v = float(r[col[metric]].replace(",", ""))
            except ValueError:
                continue
            rec[key] = v * SCALE.get(units[col[metric]], 1.0)
        out.append(rec)
    return out


def main():
    ap = argparse.ArgumentParser(description=__doc__, formatter_class=argparse.RawDescriptionHelpFormatter)
    ap.add_argument("report")
    ap.add_argument("bench_line")
    ap.add_argument("-o", "--out", required=True)
    ap.add_argument("--command", default="")
    a = ap.parse_args()
    line = None
    for raw in open(a.bench_line):
        raw = raw.strip()
        if raw.startswith("{") and '"metric"' in raw:
            line = json.loads(raw)
    if line is None:
        raise SystemExit("no bench.py JSON line in " + a.bench_line)
    units = {"request": line["requests_per_step"], "iteration": line["sim_iterations_per_step"],
             "round": line["ls_rounds_executed_per_step"]}
    kernels = {}
    for rec in read_report(a.report):
        name = rec.pop("kernel")
        if name in kernels or name not in UNIT:          # first captured launch of each kernel
            continue
        n = float(units[UNIT[name]])
        kernels[name] = dict(unit=UNIT[name], units_in_capture=n,
                             dram_bytes_per_unit=(rec.get("dram_read", 0.0) + rec.get("dram_write", 0.0)) / n,
                             warp_inst_per_unit=rec.get("warp_inst", 0.0) / n, **rec)
    doc = dict(source_hash=_build.source_hash(), workload=line["config"]["workload"], shape=line.get("shape"),
               command=a.command,
               note="one launch of each kernel; per-launch times under the profiler are cold-cache and serialised",
               kernels=kernels)
    with open(a.out, "w") as fh:
        json.dump(doc, fh, indent=1, sort_keys=True)
        fh.write("\n")
    print("wrote", a.out, "for", ", ".join(sorted(kernels)))


if __name__ == "__main__":
    main()
