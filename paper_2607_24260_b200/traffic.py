"""DRAM traffic of the attention kernel per algorithmic byte, as measured by one ncu capture, kept in
a small tracked text file together with a digest of the kernel sources it was measured on.

    python -m paper_2607_24260_b200.traffic decode <ncu raw csv> <algorithmic bytes per launch> [kernel name part]
    python -m paper_2607_24260_b200.traffic verify <ncu raw csv> <algorithmic bytes per launch> [kernel name part]

(kernel name part: which launches of the csv to average, e.g. "split_kernel<1" for the proposal
instantiation and "split_kernel<2" for the verification one; default: every kap_attn_split_kernel.)

The csv is what `ncu -i <report> --page raw --csv` prints for a capture of kap_attn_split_kernel
(`dram__bytes_read.sum` and `dram__bytes_write.sum` per launch).  The benchmark reads the file
back and reports the traffic only while the digest still matches the sources it runs: a ratio
measured on another version of the kernel is not reported.
"""
from __future__ import annotations

import csv
import glob
import hashlib
import os
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(HERE)
RATIO_FILE = os.path.join(ROOT, "profiles", "traffic_ratio.txt")
KERNEL_SOURCES = ("kap_attn_kernel.cuh", "kap_attn.cu", "kap_schedule.cpp", "kap_internal.h")


def kernel_digest() -> str:
    h = hashlib.sha256()
    for name in KERNEL_SOURCES:
        with open(os.path.join(HERE, "csrc", name), "rb") as f:
            h.update(f.read())
    return h.hexdigest()[:16]


def read_ratios() -> dict:
    """{"decode": ratio or None, "verify": ratio or None}; None when the file is missing, has no
    entry, or was written for other kernel sources."""
    out = {"decode": None, "verify": None}
    try:
        with open(RATIO_FILE) as f:
            rows = [line.split() for line in f if line.strip() and not line.startswith("#")]
    except OSError:
        return out
    now = kernel_digest()
    for row in rows:
        if len(row) >= 3 and row[0] in out and row[2] == now:
            out[row[0]] = float(row[1])
    return out


def _to_bytes(value: str, unit: str) -> float:
    scale = {"byte": 1.0, "Kbyte": 1e3, "Mbyte": 1e6, "Gbyte": 1e9}
    return float(value.replace(",", "")) * scale.get(unit, 1.0)


def traffic_from_csv(path: str, kernel_substr: str = "kap_attn_split_kernel") -> float:
    """mean over the captured launches of dram__bytes_read.sum + dram__bytes_write.sum"""
    with open(path, newline="") as f:
        rows = list(csv.reader(f))
    head = next(i for i, r in enumerate(rows) if "Kernel Name" in r)
    names, units = rows[head], rows[head + 1]
    col = {n: i for i, n in enumerate(names)}
    total, n = 0.0, 0
    for r in rows[head + 2:]:
        if len(r) < len(names) or kernel_substr not in r[col["Kernel Name"]]:
            continue
        total += sum(_to_bytes(r[col[m]], units[col[m]]) for m in ("dram__bytes_read.sum", "dram__bytes_write.sum"))
        n += 1
    if not n:
        raise SystemExit(f"no launch of {kernel_substr} in {path}")
    return total / n


def write_ratio(kind: str, ratio: float, note: str):
    keep = []
    if os.path.exists(RATIO_FILE):
        with open(RATIO_FILE) as f:
            keep = [line for line in f if line.startswith("#") or (line.split() and line.split()[0] != kind)]
    if not keep:
        keep = ["# DRAM bytes (read + write, ncu) per algorithmic byte of one kap_attn_split_kernel launch.\n",
                "# kind  ratio  digest-of-kernel-sources  note   (written by paper_2607_24260_b200/traffic.py)\n"]
    keep.append(f"{kind} {ratio:.4f} {kernel_digest()} {note}\n")
    with open(RATIO_FILE, "w") as f:
        f.writelines(keep)


if __name__ == "__main__":
    kind, path, alg = sys.argv[1], sys.argv[2], float(sys.argv[3])
    assert kind in ("decode", "verify")
    t = traffic_from_csv(path, *sys.argv[4:5])
    write_ratio(kind, t / alg, f"{t:.0f}B/{alg:.0f}B from {os.path.basename(path)}")
    print(kind, t / alg)
