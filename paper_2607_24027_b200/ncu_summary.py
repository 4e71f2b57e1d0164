"""Turn an Nsight Compute report of one of this library's kernels into the small JSON that bench.py reads.

    python -m paper_2607_24027_b200.ncu_summary REPORT.ncu-rep --kernel fwd_sm100_kernel \
        --workload video720 --heads 4 [--command "the command that was profiled"]

Reads the report with ``ncu -i REPORT --page raw --csv`` (no GPU needed), takes the first launch whose
name contains ``--kernel`` and writes ``profiles/<kernel>_<workload>.json``: DRAM bytes read and written
by that launch, its duration and the utilisation counters quoted in the summaries, together with the
head count of the captured case and the git hash of the kernel's source, so that a stale summary is
visible.  ``bench.py`` scales the DRAM bytes by the head count of the timed launch.
"""
from __future__ import annotations

import argparse
import csv
import io
import json
import os
import subprocess

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WANTED = {
    "dram_bytes_read": "dram__bytes_read.sum",
    "dram_bytes_write": "dram__bytes_write.sum",
    "duration": "gpu__time_duration.sum",
    "tensor_pipe_active_pct": "sm__pipe_tensor_cycles_active.avg.pct_of_peak_sustained_active",
    "dram_throughput_pct": "gpu__dram_throughput.avg.pct_of_peak_sustained_elapsed",
    "xu_pipe_pct": "sm__inst_executed_pipe_xu.avg.pct_of_peak_sustained_active",
    "issue_active_pct": "sm__issue_active.avg.pct_of_peak_sustained_elapsed",
    "l2_to_sm_tma_bytes": "l1tex__m_xbar2l1tex_read_bytes_mem_global_op_tma_ld.sum",
    "l2_throughput_pct": "lts__throughput.avg.pct_of_peak_sustained_elapsed",
    "warps_active": "sm__warps_active.avg.per_cycle_active",
    "registers_per_thread": "launch__registers_per_thread",
}
UNIT_SCALE = {"byte": 1.0, "Kbyte": 1e3, "Mbyte": 1e6, "Gbyte": 1e9, "Tbyte": 1e12,
              "ns": 1e-9, "us": 1e-6, "ms": 1e-3, "s": 1.0, "second": 1.0, "msecond": 1e-3, "usecond": 1e-6,
              "nsecond": 1e-9}


def read_report(path: str):
    out = subprocess.run(["ncu", "-i", path, "--page", "raw", "--csv"], capture_output=True, text=True, check=True)
    rows = list(csv.reader(io.StringIO(out.stdout)))
    header = next(i for i, r in enumerate(rows) if "Kernel Name" in r)
    names, units = rows[header], rows[header + 1]
    return names, units, rows[header + 2:]


def summarise(path: str, kernel: str):
    names, units, launches = read_report(path)
    k_col = names.index("Kernel Name")
    row = next(r for r in launches if kernel in r[k_col])
    rec = {"kernel": row[k_col].split("(")[0]}
    for key, metric in WANTED.items():
        if metric not in names:
            continue
        c = names.index(metric)
        try:
            val = float(row[c].replace(",", ""))
        except ValueError:
            continue
        rec[key] = val * UNIT_SCALE.get(units[c], 1.0)
    return rec


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("report")
    ap.add_argument("--kernel", required=True)
    ap.add_argument("--workload", required=True)
    ap.add_argument("--heads", type=int, required=True)
    ap.add_argument("--command", default="")
    a = ap.parse_args()
    rec = summarise(a.report, a.kernel)
    rec.update({"workload": a.workload, "heads": a.heads, "report": os.path.basename(a.report), "command": a.command})
    src = {"fwd_sm100_kernel": "fwd_sm100.cu", "pool_kernel": "pool.cu"}.get(a.kernel, "")
    try:
        rec["kernel_git_hash"] = subprocess.run(
            ["git", "log", "-1", "--format=%h", "--", os.path.join("paper_2607_24027_b200", "csrc", src)],
            cwd=ROOT, capture_output=True, text=True, check=True).stdout.strip()
    except Exception:
        rec["kernel_git_hash"] = None
    out = os.path.join(ROOT, "profiles", f"{a.kernel}_{a.workload}.json")
    with open(out, "w") as f:
        json.dump(rec, f, indent=1)
        f.write("\n")
    print(out, json.dumps(rec))


if __name__ == "__main__":
    main()
