"""Turn an Nsight Compute report of a libkop kernel into the short text summary kept under profiles/ and update
the table of measured DRAM traffic that bench.py reports next to each kernel's algorithmic bytes.

  python -m paper_2609_30059_b200.ncu_summary REPORT.ncu-rep --kernel ln_pair_kernel \
      --out profiles/ln_pair_kernel_bf16_8192x4096.md --workload "kop_bias_gelu_residual_layernorm, bf16 [8192,4096]" \
      --bytes 201441280 --command "ncu ... python bench.py --profile layernorm --launches 1" \
      [--segment layernorm --rows-div 1]

The report is read with `ncu -i REPORT --page raw --csv` (works on a machine without a GPU); a .csv file written by
`ncu --csv --page raw --log-file FILE` is read as it is. The LAST captured
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
    """Rows of `ncu --page raw --csv` as dicts, plus the units row. `path` is an .ncu-rep report, or the CSV that
    `ncu --csv --page raw --log-file FILE ...` wrote directly (a report embeds the whole module's machine code and
    gets large for a library with many template instances; the CSV holds the counters only)."""
    if path.endswith(".csv"):
        with open(path) as f:
            text = f.read()
    else:
        text = subprocess.run(["ncu", "-i", path, "--page", "raw", "--csv"], capture_output=True, text=True, check=True).stdout
    rows = list(csv.reader(io.StringIO(text)))
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


# kernel-name prefix -> bench.py segment, for the share comparison of the launch list (the benchmark's eight kernels)
STEP_KERNELS = {"ce_row_kernel<__nv_bfloat16, 4, 0, 0>": "ce_loss", "silu_mul_kernel<": "silu_mul",
                "softmax_warp_kernel<float, float, 4, 1, 1, 32>": "softmax_large", "residual_add_kernel<": "residual_add",
                "bn_plane_block_kernel<": "bn_pool", "rmsnorm_block_kernel<__nv_bfloat16, float, 4, 1, 1, 0>": "rmsnorm",
                "ln_pair_kernel<__nv_bfloat16, float, 2, 1, 256, 0>": "layernorm"}


def launch_list(csv_path: str, out: str, command: str, note: str = "", min_share: float = 0.0005,
                bench_json: str | None = None) -> None:
    """Summary of `ncu --metrics gpu__time_duration.sum --csv --log-file FILE <cmd>` (one pass, every launch of the
    process): per kernel its launches, total time and share of all captured launches."""
    import collections
    rows = [r for r in csv.reader(open(csv_path)) if len(r) > 5]
    header, agg = None, collections.OrderedDict()
    for r in rows:
        if r[0] == "ID":
            header = r
            continue
        if header is None:
            continue
        d = dict(zip(header, r))
        if d.get("Metric Name") != "gpu__time_duration.sum":
            continue
        name = d["Kernel Name"].split("(")[0].replace("void ", "").replace("kop::", "").replace("<unnamed>::", "")[:90]
        t_us = number(d["Metric Value"]) * TO_US.get(d.get("Metric Unit", "ns"), 1e-3)
        a = agg.setdefault(name, [0, 0.0, []])
        a[0] += 1
        a[1] += t_us
        a[2].append(t_us)
    total = sum(a[1] for a in agg.values())
    with open(out, "w") as o:
        o.write("# ncu launch list of the benchmark command\n\nCommand (run on one B200 after the same command had exited 0 "
                f"without ncu; one pass, no replay):\n\n```\n{command}\n```\n\n")
        if note:
            o.write(note + "\n\n")
        o.write("Times are cold-cache and serialised: shares are comparable with the benchmark, absolutes are not.\n\n"
                "| kernel | launches | total us | share of all | mean us |\n|---|---|---|---|---|\n")
        for k, a in sorted(agg.items(), key=lambda kv: -kv[1][1]):
            if a[1] / total >= min_share:
                o.write(f"| `{k}` | {a[0]} | {a[1]:.1f} | {100 * a[1] / total:.2f} % | {a[1] / a[0]:.1f} |\n")
        if bench_json:
            with open(bench_json) as f:
                seg = json.loads(f.read().strip().splitlines()[-1])["segments"]
            means = {}
            for k, a in agg.items():
                for prefix, nm in STEP_KERNELS.items():
                    if k.startswith(prefix):
                        big = [t for t in a[2] if t > 0.7 * max(a[2])]      # the full-size launches (others are set-up
                                                                          # or the same kernel on a smaller tensor)
                        if big:
                            means[nm] = sum(big) / len(big)
            tn, tb = sum(means.values()), sum(seg[nm]["us"] for nm in means)
            o.write("\n## Share of one fused step: ncu mean per launch against the benchmark's CUDA events\n\n"
                    f"Benchmark column: the `segments` of `{os.path.basename(bench_json)}` (`python bench.py`, same build).\n\n"
                    "| segment | ncu mean us | ncu share | bench event us | bench share |\n|---|---|---|---|---|\n")
            for nm, m in sorted(means.items(), key=lambda kv: -kv[1]):
                o.write(f"| {nm} | {m:.1f} | {100 * m / tn:.1f} % | {seg[nm]['us']} | {100 * seg[nm]['us'] / tb:.1f} % |\n")
            o.write("\nEvent times are longer than the ncu means by a launch gap (~2 us) plus the write-back of dirty L2 "
                    "lines, which ncu's cold, clean-cache launches neither inherit nor pay for.\n")


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
    ap.add_argument("--launch-list", action="store_true",
                    help="REPORT is the CSV log of a gpu__time_duration.sum pass over a whole command: write the per-kernel table")
    ap.add_argument("--bench-json", default=None, help="with --launch-list: a bench.py output file to compare shares with")
    ap.add_argument("--kernel", default=None, help="substring of the kernel name")
    ap.add_argument("--out", required=True, help="summary file to write (profiles/<kernel>_<workload>.md)")
    ap.add_argument("--workload", default="")
    ap.add_argument("--bytes", type=int, default=0, help="algorithmic bytes of the captured launch")
    ap.add_argument("--command", required=True, help="the full ncu command that produced the report")
    ap.add_argument("--segment", default=None, help="bench.py segment name whose traffic entry to update")
    ap.add_argument("--rows-div", type=int, default=1, help="the capture ran on 1/N of the benchmark's rows")
    ap.add_argument("--note", default="")
    a = ap.parse_args()
    if a.launch_list:
        launch_list(a.report, a.out, a.command, a.note, bench_json=a.bench_json)
        return
    if not a.kernel or a.bytes <= 0:
        ap.error("--kernel and --bytes are required for a kernel summary")
    print(json.dumps(summarise(a.report, a.kernel, a.out, a.workload, a.bytes, a.command, a.segment, a.rows_div, a.note)))


if __name__ == "__main__":
    main()
