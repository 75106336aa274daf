"""Turns an ncu capture into a row of ``profiles/dram_traffic.txt``.

    ncu -i capture.ncu-rep --page raw --csv > capture.csv
    python -m paper_2603_14360_b200.ncu_traffic capture.csv --workload fwd_bf16 \
        --kernel fwd_bf16_cs_kernel --source scan_fwd_bf16_cs.cu --units 262144

The row holds, for one launch of the workload's dominant kernel, the DRAM bytes the profiler
counted (dram__bytes_read.sum + dram__bytes_write.sum, averaged over the captured launches), the
token-heads (B T N; decode: B N) the captured launch processed, and a digest of the kernel's sources at capture time.
``bench.py`` reports the figure as ``roofline.traffic``, scaled to a full launch by token-heads, and
reports null once the sources have changed.  A step made of several kernels (`in_conv`, `out_norm`)
has one row per kernel, named `workload:part`; bench.py adds them.
"""
from __future__ import annotations

import argparse
import csv
import hashlib
import os
import re

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
TABLE = os.path.join(os.path.dirname(HERE), "profiles", "dram_traffic.txt")
HEADER = ("# DRAM traffic of one launch of each workload's dominant kernel, from ncu captures.\n"
          "# Written by `python -m paper_2603_14360_b200.ncu_traffic`; read by bench.py (roofline.traffic).\n"
          "# workload[:kernel of a step made of several]  kernel  source  dram_bytes_per_launch  units_captured (token-heads; tokens for in_conv, out_norm)  source_digest  ncu_dram_read  ncu_dram_write  launches\n")


def source_digest(cu_file: str) -> str:
    h = hashlib.sha256()
    for f in [cu_file] + sorted(x for x in os.listdir(CSRC) if x.endswith((".cuh", ".h"))):
        h.update(open(os.path.join(CSRC, f), "rb").read())
    return h.hexdigest()[:16]


def _to_bytes(value: str, unit: str) -> float:
    scale = {"byte": 1.0, "Kbyte": 1e3, "Mbyte": 1e6, "Gbyte": 1e9, "Tbyte": 1e12}[unit]
    return float(value.replace(",", "")) * scale


def dram_bytes(csv_path: str, kernel_regex: str):
    """(mean read bytes, mean write bytes, launches) over the rows whose kernel name matches."""
    rows = list(csv.reader(open(csv_path, newline="")))
    start = next(i for i, r in enumerate(rows) if "Kernel Name" in r)
    names, units = rows[start], rows[start + 1]
    col = {n: i for i, n in enumerate(names)}
    rd, wr = col["dram__bytes_read.sum"], col["dram__bytes_write.sum"]
    reads, writes = [], []
    for r in rows[start + 2:]:
        if len(r) <= max(rd, wr) or not re.search(kernel_regex, r[col["Kernel Name"]]):
            continue
        reads.append(_to_bytes(r[rd], units[rd]))
        writes.append(_to_bytes(r[wr], units[wr]))
    if not reads:
        raise SystemExit(f"no launch of a kernel matching {kernel_regex!r} in {csv_path}")
    return sum(reads) / len(reads), sum(writes) / len(writes), len(reads)


def main():
    ap = argparse.ArgumentParser(description=__doc__, formatter_class=argparse.RawDescriptionHelpFormatter)
    ap.add_argument("csv")
    ap.add_argument("--workload", required=True)
    ap.add_argument("--kernel", required=True, help="regular expression matched against the kernel name")
    ap.add_argument("--source", required=True, help="the kernel's .cu file under csrc/")
    ap.add_argument("--units", type=int, required=True, help="token-heads the captured launch processed")
    a = ap.parse_args()
    rd, wr, n = dram_bytes(a.csv, a.kernel)
    row = f"{a.workload}  {a.kernel}  {a.source}  {rd + wr:.6g}  {a.units}  {source_digest(a.source)}  {rd:.6g}  {wr:.6g}  {n}\n"
    old = [ln for ln in open(TABLE)] if os.path.exists(TABLE) else []
    keep = [ln for ln in old if not ln.startswith("#") and ln.split() and ln.split()[0] != a.workload]
    with open(TABLE, "w") as f:
        f.write(HEADER)
        f.writelines(sorted(keep + [row]))
    print(row, end="")


if __name__ == "__main__":
    main()
