"""Turn the raw CSV page of an ncu report into the small counter file the benchmark quotes.

    ncu -i <capture>.ncu-rep --page raw --csv > raw.csv
    python -m paper_2603_11021_b200.ncu_counters raw.csv profiles/<name>_counters.json --blocks <blocks per launch>

The counter file records, beside the counters of the first captured launch, the names and the hash of the sources the
captured kernel is compiled from at the time it is written (write it from the tree the capture ran on).  ``bench.py`` prints the counters only while
that hash still matches the sources it runs: a kernel edited after its capture gets no stale numbers.
"""
from __future__ import annotations

import argparse
import csv
import glob
import hashlib
import json
import os
import subprocess

PKG = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(PKG)

KEYS = {
    "gpu__time_duration.sum": "duration_ns",
    "dram__bytes_read.sum": "dram_bytes_read",
    "dram__bytes_write.sum": "dram_bytes_write",
    "smsp__inst_executed.sum": "warp_instructions",
    "smsp__issue_active.avg.pct_of_peak_sustained_active": "issue_active_pct",
    "sm__inst_executed_pipe_alu.avg.pct_of_peak_sustained_active": "pipe_alu_pct",
    "sm__inst_executed_pipe_fma.avg.pct_of_peak_sustained_active": "pipe_fma_pct",
    "sm__inst_executed_pipe_lsu.avg.pct_of_peak_sustained_active": "pipe_lsu_pct",
    "sm__pipe_tensor_cycles_active.avg.pct_of_peak_sustained_active": "pipe_tensor_pct",
    "l1tex__data_pipe_lsu_wavefronts_mem_shared.sum": "shared_wavefronts",
    "l1tex__data_bank_conflicts_pipe_lsu_mem_shared.sum": "shared_bank_conflicts",
    "launch__registers_per_thread": "registers_per_thread",
    "sm__cycles_active.avg": "sm_cycles_active",
    "sm__cycles_elapsed.avg": "sm_cycles_elapsed",
}

_SCALE = {"byte": 1.0, "Kbyte": 1e3, "Mbyte": 1e6, "Gbyte": 1e9, "ns": 1.0, "us": 1e3, "ms": 1e6, "s": 1e9, "usecond": 1e3, "nsecond": 1.0,
          "msecond": 1e6, "second": 1e9}


# what the fused GEMV kernels are compiled from (the default set of sources a counter file vouches for)
GEMV_SOURCES = ["tables.h", "tables.cpp", "ctx.h", "decode.cuh", "fast.cuh", "big.cuh", "umma.cuh", "kernels_common.cuh", "gemv_kernels.cuh",
                "gemv.cu"]


def source_hash(names=None) -> str:
    """SHA-256 over the named files under csrc (default: everything there), in a fixed order."""
    h = hashlib.sha256()
    files = sorted(glob.glob(os.path.join(PKG, "csrc", "*"))) if names is None else [os.path.join(PKG, "csrc", n) for n in sorted(names)]
    for f in files:
        h.update(os.path.basename(f).encode())
        with open(f, "rb") as fh:
            h.update(fh.read())
    return h.hexdigest()[:16]


def load(path: str) -> dict | None:
    """The counter file, or None when it is missing or the sources it names have changed since it was written."""
    try:
        with open(path) as f:
            d = json.load(f)
        return d if d.get("source_hash") == source_hash(d.get("sources")) else None
    except (OSError, ValueError):
        return None


def parse_raw_csv(path: str, kernel_filter: str | None = None) -> dict:
    with open(path, newline="") as f:
        rows = list(csv.reader(f))
    hdr, units = rows[0], rows[1]
    name_col = hdr.index("Kernel Name")
    for r in rows[2:]:
        if kernel_filter and kernel_filter not in r[name_col]:
            continue
        out = {"kernel": r[name_col].split("(")[0]}
        for i, h in enumerate(hdr):
            if h in KEYS and r[i] not in ("", "n/a"):
                out[KEYS[h]] = float(r[i].replace(",", "")) * _SCALE.get(units[i], 1.0)
        return out
    raise SystemExit("no matching kernel in " + path)


def main() -> None:
    ap = argparse.ArgumentParser()
    ap.add_argument("raw_csv")
    ap.add_argument("out_json")
    ap.add_argument("--kernel", default=None, help="substring of the kernel name to pick (default: the first launch)")
    ap.add_argument("--blocks", type=int, required=True, help="blocks of 24 weights one launch processes")
    ap.add_argument("--workload", default="")
    ap.add_argument("--sources", nargs="*", default=GEMV_SOURCES, help="files under csrc the captured kernel is compiled from")
    args = ap.parse_args()
    c = parse_raw_csv(args.raw_csv, args.kernel)
    c["blocks_per_launch"] = args.blocks
    c["workload"] = args.workload
    c["sources"] = sorted(args.sources)
    c["source_hash"] = source_hash(args.sources)
    try:
        c["git_commit"] = subprocess.check_output(["git", "-C", ROOT, "rev-parse", "--short", "HEAD"], text=True).strip()
    except Exception:
        c["git_commit"] = None
    if "warp_instructions" in c:
        c["warp_instructions_per_block"] = c["warp_instructions"] / args.blocks
        c["thread_instructions_per_block"] = 32.0 * c["warp_instructions"] / args.blocks     # one lane decodes one block
    if "shared_wavefronts" in c:
        c["shared_wavefronts_per_32_blocks"] = 32.0 * c["shared_wavefronts"] / args.blocks
    if "dram_bytes_read" in c:
        c["dram_traffic_bytes"] = c["dram_bytes_read"] + c.get("dram_bytes_write", 0.0)
    with open(args.out_json, "w") as f:
        json.dump(c, f, indent=1, sort_keys=True)
        f.write("\n")
    print(json.dumps(c))


if __name__ == "__main__":
    main()
