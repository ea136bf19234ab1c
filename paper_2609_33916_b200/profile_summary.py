"""Reads an Nsight Compute report (`ncu -i <file>.ncu-rep --page raw --csv`) and prints the counters the
roofline entries of bench.py rest on, one block per captured launch; with --record it also writes the
measured DRAM traffic of a kernel into profiles/traffic.json, the record bench.py scales by tokens for
`roofline.traffic` (so that the bench line never carries a number typed in by hand).

    python -m paper_2609_33916_b200.profile_summary prof_bwd.ncu-rep \\
        --record bwd_kv --case "B1 H8 n8192 d128 non-causal, TMA bulk reduce" --tokens 65536 --d 128 --dq-mode 2

No GPU is needed to read a report.  Nothing here is on the product path.
"""
from __future__ import annotations

import argparse
import csv
import json
import os
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

COUNTERS = [
    "gpu__time_duration.sum", "dram__bytes_read.sum", "dram__bytes_write.sum",
    "gpu__dram_throughput.avg.pct_of_peak_sustained_elapsed",
    "sm__pipe_tensor_cycles_active.avg.pct_of_peak_sustained_active",
    "sm__pipe_tensor_cycles_active.avg.pct_of_peak_sustained_elapsed",
    "sm__warps_active.avg.pct_of_peak_sustained_active", "smsp__issue_active.avg.pct_of_peak_sustained_active",
    "sm__inst_executed_pipe_xu.sum.pct_of_peak_sustained_active", "smsp__inst_executed_op_global_red.sum",
    "l1tex__data_bank_conflicts_pipe_lsu_mem_shared.sum", "lts__throughput.avg.pct_of_peak_sustained_elapsed",
    "launch__registers_per_thread", "launch__grid_size", "launch__block_size", "launch__waves_per_multiprocessor",
    "launch__cluster_x",
]


def read_report(path: str) -> list[dict]:
    out = subprocess.run(["ncu", "-i", path, "--page", "raw", "--csv"], capture_output=True, text=True, check=True).stdout
    rows = list(csv.reader(out.splitlines()))
    hdr, units = rows[0], rows[1]
    launches = []
    for r in rows[2:]:
        d = {h: (r[i], units[i]) for i, h in enumerate(hdr) if i < len(r)}
        launches.append(d)
    return launches


def to_bytes(value: str, unit: str) -> float:
    v = float(value.replace(",", ""))
    scale = {"byte": 1.0, "Kbyte": 1e3, "Mbyte": 1e6, "Gbyte": 1e9}
    return v * scale.get(unit, 1.0)


def main() -> int:
    ap = argparse.ArgumentParser()
    ap.add_argument("report")
    ap.add_argument("--record", default="", help="kernel kind (fwd, bwd_kv, bwd_dq) to record DRAM traffic for")
    ap.add_argument("--case", default="")
    ap.add_argument("--tokens", type=int, default=0, help="B*H*n of the captured case")
    ap.add_argument("--d", type=int, default=128)
    ap.add_argument("--dq-mode", type=int, default=2)
    ap.add_argument("--causal", type=int, default=0)
    ap.add_argument("--launch", type=int, default=0, help="which captured launch to record")
    ap.add_argument("--command", default="", help="the command line that produced the report (kept in the record)")
    args = ap.parse_args()
    launches = read_report(args.report)
    for i, d in enumerate(launches):
        name = d.get("Kernel Name", ("", ""))[0]
        print(f"launch {i}: {name[:90]}")
        for c in COUNTERS:
            if c in d:
                print(f"  {c} [{d[c][1]}] = {d[c][0]}")
    if args.record:
        d = launches[args.launch]
        total = to_bytes(*d["dram__bytes_read.sum"]) + to_bytes(*d["dram__bytes_write.sum"])
        path = os.path.join(ROOT, "profiles", "traffic.json")
        try:
            with open(path) as f:
                rec = json.load(f)
        except Exception:
            rec = {}
        rec[args.record] = {
            "kernel": d.get("Kernel Name", ("", ""))[0], "case": args.case, "tokens": args.tokens,
            "dram_bytes_per_launch": total, "dram_bytes_read": to_bytes(*d["dram__bytes_read.sum"]),
            "dram_bytes_written": to_bytes(*d["dram__bytes_write.sum"]),
            "family": {"d": args.d, "causal": bool(args.causal), "dq_mode": args.dq_mode},
            "command": args.command,
        }
        with open(path, "w") as f:
            json.dump(rec, f, indent=1, sort_keys=True)
            f.write("\n")
        print(f"recorded {args.record}: {total / 1e6:.1f} MB per launch over {args.tokens} tokens -> {path}")
    return 0


if __name__ == "__main__":
    sys.exit(main())
