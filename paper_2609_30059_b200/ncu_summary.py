"""Turn an Nsight Compute report of a libkop kernel into the short text summary kept under profiles/ and update
the table of measured DRAM traffic that bench.py reports next to each kernel's algorithmic bytes.

  python -m paper_2609_30059_b200.ncu_summary REPORT.ncu-rep --kernel ln_pair_kernel \
      --out profiles/ln_pair_kernel_bf16_8192x4096.md --workload "kop_bias_gelu_residual_layernorm, bf16 [8192,4096]" \
      --bytes 201441280 --command "ncu ... python bench.py --profile layernorm --launches 1" \
      [--segment layernorm --rows-div 1]

The report is read with `ncu -i REPORT --page raw --csv` (works on a machine without a GPU). The LAST captured
launch whose kernel name contains --kernel is summarised (the first is usually a warm-up launch). With --segment,
profiles/ncu_dram_traffic.json gets that segment's dram read / write bytes, the capture's row divisor (a capture on
1/N of the benchmark's rows, whose traffic is proportional to rows) and the name of the summary it came from;
bench.py reads that file, so the figures it prints cannot drift from the committed summaries.
"""
from __future__ import annotations

import argparse
import csv
import io
import json
import os
import subprocess

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
TRAFFIC_FILE = os.path.join(ROOT, "profiles", "ncu_dram_traffic.json")

METRICS = [
    ("gpu__time_duration.sum", "duration (ncu, cold caches, serialised)"),
    ("dram__bytes_read.sum", "DRAM bytes read"),
    ("dram__bytes_write.sum", "DRAM bytes written (dirty lines still in L2 at kernel end are not counted)"),
    ("gpu__dram_throughput.avg.pct_of_peak_sustained_elapsed", "DRAM throughput, % of ncu peak"),
    ("sm__throughput.avg.pct_of_peak_sustained_elapsed", "SM throughput %"),
    ("l1tex__throughput.avg.pct_of_peak_sustained_active", "L1/TEX throughput %"),
    ("lts__throughput.avg.pct_of_peak_sustained_elapsed", "L2 throughput %"),
    ("smsp__issue_active.avg.pct_of_peak_sustained_active", "issue slots busy %"),
    ("sm__inst_executed_pipe_xu.avg.pct_of_peak_sustained_active", "XU (MUFU) pipe %"),
    ("sm__inst_executed_pipe_fma.avg.pct_of_peak_sustained_active", "FMA pipe %"),
    ("sm__inst_executed_pipe_alu.avg.pct_of_peak_sustained_active", "ALU pipe %"),
    ("sm__warps_active.avg.pct_of_peak_sustained_active", "achieved occupancy %"),
    ("launch__registers_per_thread", "registers / thread"),
    ("launch__block_size", "block size"),
    ("launch__grid_size", "grid size"),
    ("launch__occupancy_limit_registers", "CTAs/SM allowed by registers"),
    ("launch__occupancy_limit_shared_mem", "CTAs/SM allowed by shared memory"),
    ("smsp__average_warps_issue_stalled_long_scoreboard_per_issue_active.ratio", "long-scoreboard stall (warps per issue)"),
    ("smsp__average_warps_issue_stalled_barrier_per_issue_active.ratio", "barrier stall (warps per issue)"),
    ("smsp__average_warps_issue_stalled_lg_throttle_per_issue_active.ratio", "LG-throttle stall (warps per issue)"),
    ("smsp__average_warps_issue_stalled_math_pipe_throttle_per_issue_active.ratio", "math-pipe-throttle stall (warps per issue)"),
]

TO_BYTES = {"byte": 1.0, "Kbyte": 1e3, "Mbyte": 1e6, "Gbyte": 1e9}
TO_US = {"ns": 1e-3, "us": 1.0, "ms": 1e3, "s": 1e6}


def read_report(path: str):
    """Rows of `ncu --page raw --csv` as dicts, plus the units row."""
    res = subprocess.run(["ncu", "-i", path, "--page", "raw", "--csv"], capture_output=True, text=True, check=True)
    rows = list(csv.reader(io.StringIO(res.stdout)))
    start = next(i for i, r in enumerate(rows) if r and r[0] == "ID")
    header, units = rows[start], rows[start + 1]
    return [dict(zip(header, r)) for r in rows[start + 2:] if len(r) == len(header)], dict(zip(header, units))


def number(text: str) -> float:
    return float(text.replace(",", ""))


def summarise(report: str, kernel: str, out: str, workload: str, nbytes: int, command: str,
              segment: str | None = None, rows_div: int = 1, note: str = "") -> dict:
    launches, units = read_report(report)
    mine = [d for d in launches if kernel in d["Kernel Name"]]
    if not mine:
        raise SystemExit(f"no captured launch whose kernel name contains {kernel!r}")
    d = mine[-1]
    dur_us = number(d["gpu__time_duration.sum"]) * TO_US[units["gpu__time_duration.sum"]]
    rd = number(d["dram__bytes_read.sum"]) * TO_BYTES[units["dram__bytes_read.sum"]]
    wr = number(d["dram__bytes_write.sum"]) * TO_BYTES[units["dram__bytes_write.sum"]]
    name = d["Kernel Name"].split("(")[0].replace("void ", "").replace("kop::", "").replace("<unnamed>::", "")
    with open(out, "w") as o:
        o.write(f"# ncu summary: `{name}`\n\nWorkload: {workload}.\n\n")
        o.write("Command (run on one B200 after the same command had exited 0 without ncu):\n\n```\n"
                f"{command}\nncu -i <report> --page raw --csv\n```\n\n")
        o.write(f"Last of {len(mine)} captured launch(es) of this kernel:\n\n| metric | value |\n|---|---|\n")
        for key, label in METRICS:
            if key in d and d[key] != "":
                o.write(f"| {label} (`{key}`) | {d[key]} {units.get(key, '')} |\n")
        o.write(f"| algorithmic bytes of this launch | {nbytes} |\n")
        o.write(f"| DRAM traffic / algorithmic bytes | {(rd + wr) / nbytes:.3f} |\n")
        o.write(f"| algorithmic GB/s at the ncu duration | {nbytes / dur_us / 1e3:.0f} |\n")
        if note:
            o.write(f"\n{note}\n")
        o.write("\nncu durations are cold-cache and serialised, and exclude the write-back of the dirty lines the "
                "kernel leaves in L2; the benchmark's CUDA-event times (bench.py) are the reported numbers.\n")
    entry = {"kernel": kernel, "summary": os.path.basename(out), "dram_read_bytes": int(round(rd)),
             "dram_write_bytes": int(round(wr)), "rows_div": int(rows_div), "ncu_duration_us": round(dur_us, 3)}
    if segment:
        table = load_traffic()
        table[segment] = entry
        with open(TRAFFIC_FILE, "w") as f:
            json.dump(table, f, indent=1, sort_keys=True)
            f.write("\n")
    return entry


def load_traffic() -> dict:
    """The committed table: segment -> measured DRAM bytes of one captured launch (see the module docstring)."""
    try:
        with open(TRAFFIC_FILE) as f:
            return json.load(f)
    except FileNotFoundError:
        return {}


def traffic_per_full_launch(segment: str):
    """dram read + write bytes of one launch at the benchmark shape (the capture scaled by its row divisor), or None."""
    e = load_traffic().get(segment)
    return None if e is None else (e["dram_read_bytes"] + e["dram_write_bytes"]) * e["rows_div"]


def main():
    ap = argparse.ArgumentParser(description=__doc__, formatter_class=argparse.RawDescriptionHelpFormatter)
    ap.add_argument("report")
    ap.add_argument("--kernel", required=True, help="substring of the kernel name")
    ap.add_argument("--out", required=True, help="summary file to write (profiles/<kernel>_<workload>.md)")
    ap.add_argument("--workload", required=True)
    ap.add_argument("--bytes", type=int, required=True, help="algorithmic bytes of the captured launch")
    ap.add_argument("--command", required=True, help="the full ncu command that produced the report")
    ap.add_argument("--segment", default=None, help="bench.py segment name whose traffic entry to update")
    ap.add_argument("--rows-div", type=int, default=1, help="the capture ran on 1/N of the benchmark's rows")
    ap.add_argument("--note", default="")
    a = ap.parse_args()
    print(json.dumps(summarise(a.report, a.kernel, a.out, a.workload, a.bytes, a.command, a.segment, a.rows_div, a.note)))


if __name__ == "__main__":
    main()
