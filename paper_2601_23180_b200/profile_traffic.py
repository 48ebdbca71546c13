"""Tracked record of measured DRAM traffic per kernel launch (the `traffic` field of the roofline).

`profiles/dram_traffic.json` holds, per (kernel, workload), the sum of the profiler's
`dram__bytes_read.sum` and `dram__bytes_write.sum` for one launch, together with a digest of the
kernel's source files at the time of the capture. `lookup` returns the figure only while those
sources are unchanged: once a kernel has been edited its old counters say nothing, and the
benchmark prints null until the capture is refreshed.

Refreshing a record (after `ncu -i capture.ncu-rep --page raw --csv > raw.csv`):

    python -m paper_2601_23180_b200.profile_traffic --csv raw.csv --kernel lmhead_gemm_kernel \
        --workload long_paged --summary profiles/lmhead_gemm_kernel_long_paged.md [--scale 4.0]

`--scale` multiplies the captured bytes when the capture ran a reduced copy of the workload whose
traffic grows in proportion to the units processed (the summary has to say so).
"""
from __future__ import annotations

import argparse
import csv
import hashlib
import json
import os
from typing import Optional

PKG = os.path.dirname(os.path.abspath(__file__))
RECORD = os.path.join(PKG, "..", "profiles", "dram_traffic.json")

# the files whose contents decide what a kernel does on the device
_COMMON = ["csrc/sm100.cuh", "csrc/host_common.h"]
SOURCES = {
    "lmhead_gemm_kernel": ["csrc/lmhead.cu"] + _COMMON,
    "lmhead_rows_kernel": ["csrc/lmhead.cu"] + _COMMON,
    "verify_attn_split_kernel": ["csrc/attn.cu", "csrc/attn_common.cuh"] + _COMMON,
    "verify_attn_pieces_kernel": ["csrc/attn_pieces.cu", "csrc/attn_common.cuh"] + _COMMON,
    "accept_scan_kernel": ["csrc/accept_scan.cu", "csrc/host_common.h"],
    "tree_mask_block_kernel": ["csrc/tree_mask.cu", "csrc/host_common.h"],
}

_UNIT = {"byte": 1.0, "Kbyte": 1e3, "Mbyte": 1e6, "Gbyte": 1e9, "Tbyte": 1e12}


def digest(kernel: str) -> str:
    h = hashlib.sha256()
    for rel in SOURCES[kernel]:
        with open(os.path.join(PKG, rel), "rb") as f:
            h.update(f.read())
    return h.hexdigest()


def _load() -> dict:
    if not os.path.exists(RECORD):
        return {}
    with open(RECORD) as f:
        return json.load(f)


def lookup(kernel: str, workload: str) -> Optional[float]:
    rec = _load().get(kernel, {}).get(workload)
    if rec is None or kernel not in SOURCES or rec.get("digest") != digest(kernel):
        return None
    return float(rec["dram_bytes_per_launch"])


def _bytes_per_launch(csv_path: str, kernel: str) -> tuple:
    """Mean over the captured launches of `kernel` of dram read + write bytes, from ncu's raw CSV page
    (a header row with the metric names, a row with their units, then one row per launch)."""
    with open(csv_path, newline="") as f:
        rows = [r for r in csv.reader(f) if r]
    hdr = next(i for i, r in enumerate(rows) if "Kernel Name" in r)
    names, units = rows[hdr], rows[hdr + 1]
    kcol = names.index("Kernel Name")
    rd, wr = names.index("dram__bytes_read.sum"), names.index("dram__bytes_write.sum")
    vals = []
    for r in rows[hdr + 2:]:
        if len(r) <= max(kcol, rd, wr) or kernel not in r[kcol]:
            continue
        vals.append(float(r[rd].replace(",", "")) * _UNIT[units[rd]] + float(r[wr].replace(",", "")) * _UNIT[units[wr]])
    if not vals:
        raise SystemExit(f"no launch of {kernel} in {csv_path}")
    return sum(vals) / len(vals), len(vals)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--csv", required=True)
    ap.add_argument("--kernel", required=True, choices=sorted(SOURCES))
    ap.add_argument("--workload", required=True)
    ap.add_argument("--summary", required=True, help="the profiles/*.md file that describes the capture")
    ap.add_argument("--scale", type=float, default=1.0)
    a = ap.parse_args()
    byts, n = _bytes_per_launch(a.csv, a.kernel)
    rec = _load()
    rec.setdefault(a.kernel, {})[a.workload] = {
        "dram_bytes_per_launch": byts * a.scale, "captured_launches": n, "scale": a.scale,
        "summary": a.summary, "digest": digest(a.kernel), "sources": SOURCES[a.kernel]}
    with open(RECORD, "w") as f:
        json.dump(rec, f, indent=1, sort_keys=True)
        f.write("\n")
    print(f"{a.kernel} on {a.workload}: {byts * a.scale / 1e6:.1f} MB per launch ({n} launches)")


if __name__ == "__main__":
    main()
