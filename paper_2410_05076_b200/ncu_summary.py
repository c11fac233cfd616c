"""Extract the DRAM traffic per kernel launch from an ncu capture of `bench.py --profile-case`.

    ncu -i capture.ncu-rep --page raw --csv > capture.csv
    python -m paper_2410_05076_b200.ncu_summary cfg3 capture.csv >> profiles/ncu_dram_traffic.txt

Prints one line per kernel, `<workload> <kernel> <bytes>`, where bytes is the mean over the captured
launches of dram__bytes_read.sum + dram__bytes_write.sum and kernel is one of full, select (the fused
selection kernel), score and value (the two passes a selection layer runs as inside a step), topk, sparse.
bench.py reads these lines for the `traffic` fields of its roofline block.
"""
from __future__ import annotations

import csv
import sys

UNIT = {"byte": 1.0, "Kbyte": 1e3, "Mbyte": 1e6, "Gbyte": 1e9}


def kernel_key(name: str):
    if "attn_kernel<0" in name or "attn_kernel<(int)0" in name:
        return "full"
    if "attn_kernel<1" in name or "attn_kernel<(int)1" in name:
        return "select"
    if "attn_kernel<2" in name or "attn_kernel<(int)2" in name:
        return "sparse"
    if "score_pass" in name:
        return "score"
    if "value_pass" in name:
        return "value"
    if "topk" in name:
        return "topk"
    return None


def main(argv):
    workload, path = argv[1], argv[2]
    with open(path, newline="") as f:
        rows = list(csv.reader(f))
    start = next(i for i, r in enumerate(rows) if r and r[0] == "ID")
    header, units = rows[start], rows[start + 1]
    col = {h: i for i, h in enumerate(header)}
    rd, wr, kn = col["dram__bytes_read.sum"], col["dram__bytes_write.sum"], col["Kernel Name"]
    acc = {}
    for r in rows[start + 2:]:
        if len(r) <= max(rd, wr):
            continue
        key = kernel_key(r[kn])
        if key is None:
            continue
        b = float(r[rd]) * UNIT[units[rd]] + float(r[wr]) * UNIT[units[wr]]
        acc.setdefault(key, []).append(b)
    for key in ("full", "select", "score", "value", "topk", "sparse"):
        if key in acc:
            print(f"{workload} {key} {sum(acc[key]) / len(acc[key]):.0f}")


if __name__ == "__main__":
    main(sys.argv)
