"""Turns Nsight Compute output for this library's kernels into the short tables kept under profiles/.

    # launch list (ncu --metrics gpu__time_duration.sum --csv --log-file launches.csv <cmd>)
    python -m paper_2604_18117_b200.ncu_summary launches launches.csv

    # one or more captured launches (ncu --set full ... -o prof <cmd>;  ncu -i prof.ncu-rep --page raw --csv > prof.csv)
    python -m paper_2604_18117_b200.ncu_summary full prof.csv

    # DRAM bytes of the GEMM launches of one captured step, as the record bench.py reads for roofline.traffic
    python -m paper_2604_18117_b200.ncu_summary traffic prof.csv --kernel lq_gemm_kernel --out profiles/gemm_dram_traffic.json \
        --command "<the ncu command line>"

Only reads files; runs nothing on a GPU.
"""
from __future__ import annotations

import argparse
import csv
import hashlib
import json
import os
import re
from collections import OrderedDict

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
CSRC = os.path.join(ROOT, "paper_2604_18117_b200", "csrc")
# source files a GEMM kernel is compiled from: a record made for other sources is stale
KERNEL_SOURCES = {"lq_gemm_kernel": ("lq_gemm.cu", "lq_device.cuh"), "lq_gemm_mx_kernel": ("lq_gemm_mx.cu", "lq_device.cuh")}


def sources_sha256(kernel: str) -> str:
    h = hashlib.sha256()
    for f in KERNEL_SOURCES[kernel]:
        h.update(open(os.path.join(CSRC, f), "rb").read())
    return h.hexdigest()


def short_name(name: str) -> str:
    name = re.sub(r"\(.*$", "", name)                       # drop the argument list
    name = name.replace("void ", "").replace("<unnamed>::", "")
    if "FillFunctor" in name:
        return "torch fill (L2 flush)"
    if "elementwise" in name or name.startswith("at::"):
        return "torch elementwise"
    return name


def rows_of(path):
    with open(path, newline="") as f:
        lines = [l for l in f if not l.startswith("==")]
    return list(csv.reader(lines))


def cmd_launches(args):
    rows = rows_of(args.csv)
    head = rows[0]
    k, m, v = head.index("Kernel Name"), head.index("Metric Name"), head.index("Metric Value")
    tot = OrderedDict()
    for r in rows[1:]:
        if len(r) <= v or r[m] != "gpu__time_duration.sum":
            continue
        n = short_name(r[k])
        c = tot.setdefault(n, [0, 0.0])
        c[0] += 1
        c[1] += float(r[v].replace(",", "")) / 1e3
    s = sum(t for _, t in tot.values())
    print("| kernel | launches | total us | share |\n|---|---|---|---|")
    for n, (c, t) in sorted(tot.items(), key=lambda kv: -kv[1][1]):
        print(f"| {n} | {c} | {t:.1f} | {100 * t / s:.1f} % |")


FULL_COLS = [("us", "gpu__time_duration.sum", 1.0), ("DRAM rd MB", "dram__bytes_read.sum", None),
             ("DRAM wr MB", "dram__bytes_write.sum", None), ("DRAM %", "gpu__dram_throughput.avg.pct_of_peak_sustained_elapsed", 1.0),
             ("L2 %", "lts__throughput.avg.pct_of_peak_sustained_elapsed", 1.0),
             ("tensor %", "sm__pipe_tensor_cycles_active.avg.pct_of_peak_sustained_elapsed", 1.0),
             ("FMA %", "sm__pipe_fma_cycles_active.avg.pct_of_peak_sustained_elapsed", 1.0),
             ("issue %", "sm__issue_active.avg.pct_of_peak_sustained_elapsed", 1.0),
             ("warps act %", "sm__warps_active.avg.pct_of_peak_sustained_active", 1.0),
             ("regs", "launch__registers_per_thread", 1.0), ("grid", "launch__grid_size", 1.0)]
UNIT_TO_MB = {"byte": 1e-6, "Kbyte": 1e-3, "Mbyte": 1.0, "Gbyte": 1e3}
UNIT_TO_US = {"ns": 1e-3, "us": 1.0, "ms": 1e3, "s": 1e6}


def launches_of(path):
    rows = rows_of(path)
    head, units = rows[0], rows[1]
    out = []
    for r in rows[2:]:
        if len(r) < len(head):
            continue
        d = {"name": short_name(r[head.index("Kernel Name")])}
        for label, metric, _ in FULL_COLS:
            if metric not in head:
                d[label] = None
                continue
            i = head.index(metric)
            x = float(r[i].replace(",", "")) if r[i] not in ("", "n/a") else None
            if x is not None and label.startswith("DRAM") and label.endswith("MB"):
                x *= UNIT_TO_MB[units[i]]
            if x is not None and label == "us":
                x *= UNIT_TO_US[units[i]]
            d[label] = x
        out.append(d)
    return out


def cmd_full(args):
    ls = launches_of(args.csv)
    labels = [l for l, _, _ in FULL_COLS]
    print("| kernel | " + " | ".join(labels) + " |\n|---|" + "---|" * len(labels))
    for d in ls:
        cells = []
        for l in labels:
            x = d[l]
            cells.append("-" if x is None else (f"{x:.0f}" if l in ("regs", "grid") else f"{x:.1f}"))
        print(f"| {d['name']} | " + " | ".join(cells) + " |")


def cmd_traffic(args):
    ls = [d for d in launches_of(args.csv) if d["name"].startswith(args.kernel)]
    if not ls:
        raise SystemExit(f"no launch of {args.kernel} in {args.csv}")
    rec = {"kernel": args.kernel, "sources_sha256": sources_sha256(args.kernel),
           "launches": len(ls),
           "dram_bytes_per_step": int(round(sum((d["DRAM rd MB"] + d["DRAM wr MB"]) for d in ls) * 1e6)),
           "per_launch_MB_read_write": [[round(d["DRAM rd MB"], 3), round(d["DRAM wr MB"], 3)] for d in ls],
           "note": "dram__bytes_read.sum + dram__bytes_write.sum of the GEMM launches of one captured step; ncu flushes the caches "
                   "before each replay and most of an output is still in the 126 MB L2 when its launch ends, so writes are under-counted",
           "command": args.command}
    with open(args.out, "w") as f:
        json.dump(rec, f, indent=1)
    print(json.dumps(rec, indent=1))


def main():
    ap = argparse.ArgumentParser()
    sub = ap.add_subparsers(dest="what", required=True)
    a = sub.add_parser("launches"); a.add_argument("csv"); a.set_defaults(fn=cmd_launches)
    a = sub.add_parser("full"); a.add_argument("csv"); a.set_defaults(fn=cmd_full)
    a = sub.add_parser("traffic"); a.add_argument("csv"); a.add_argument("--kernel", required=True)
    a.add_argument("--out", required=True); a.add_argument("--command", default=""); a.set_defaults(fn=cmd_traffic)
    args = ap.parse_args()
    args.fn(args)


if __name__ == "__main__":
    main()
