"""Turns Nsight Compute output into the short text summaries kept under profiles/ (host-side text processing only).

    python -m paper_2605_07355_b200.ncu_summary launches  <launch list .csv>
    python -m paper_2605_07355_b200.ncu_summary metrics   <metrics .csv>          (per launch: the metrics asked for)
    python -m paper_2605_07355_b200.ncu_summary full      <raw page .csv>          (ncu -i x.ncu-rep --page raw --csv)
    python -m paper_2605_07355_b200.ncu_summary traffic   <raw page .csv> <workload> <out .json>

`traffic` writes the DRAM bytes per launch of each kernel kind next to the hash of the sources they were taken on;
bench.py reports them as roofline.traffic only while that hash still matches the library it runs.
"""
from __future__ import annotations

import csv
import json
import sys
from collections import OrderedDict, defaultdict

from . import accounting

KINDS = [("k_norm_sum", "norm_sum"), ("k_frame_stats", "frame_stats"), ("k_match", "match"), ("k_compact", "compact")]

FULL_KEYS = [
    "gpu__time_duration.sum", "dram__bytes_read.sum", "dram__bytes_write.sum",
    "gpu__dram_throughput.avg.pct_of_peak_sustained_elapsed", "lts__t_sector_op_read_hit_rate.pct",
    "lts__throughput.avg.pct_of_peak_sustained_elapsed", "l1tex__throughput.avg.pct_of_peak_sustained_active",
    "sm__warps_active.avg.pct_of_peak_sustained_active", "smsp__issue_active.avg.pct_of_peak_sustained_active",
    "sm__pipe_tensor_cycles_active.avg.pct_of_peak_sustained_active",
    "sm__inst_executed_pipe_uniform.avg.pct_of_peak_sustained_active", "launch__registers_per_thread",
    "launch__grid_size", "launch__block_size", "launch__cluster_size", "launch__shared_mem_per_block_dynamic",
    "launch__occupancy_limit_shared_mem", "sm__cycles_active.avg", "gpc__cycles_elapsed.max",
]


def kind_of(name: str) -> str:
    for prefix, kind in KINDS:
        if prefix in name:
            return kind
    return "other"


def short(name: str) -> str:
    return name.split("(")[0].replace("void ", "").replace("ttf::", "")[:44]


def read_long(path):
    """csv with one row per (launch, metric): returns OrderedDict[(id, kernel)] -> {metric: (value, unit)}"""
    rows = [r for r in csv.reader(open(path)) if len(r) > 8]
    hdr = rows[0]
    ki, mi, vi, ui, ii = (hdr.index(k) for k in ("Kernel Name", "Metric Name", "Metric Value", "Metric Unit", "ID"))
    out = OrderedDict()
    for r in rows[1:]:
        out.setdefault((int(r[ii]), r[ki]), {})[r[mi]] = (r[vi].replace(",", ""), r[ui])
    return out


def read_wide(path):
    """csv of `--page raw`: one row per launch, one column per metric; second row holds the units"""
    rows = [r for r in csv.reader(open(path)) if len(r) > 8]
    hdr, units = rows[0], rows[1]
    ki = hdr.index("Kernel Name")
    out = []
    for r in rows[2:]:
        out.append((r[ki], {h: (v.replace(",", ""), u) for h, v, u in zip(hdr, r, units)}))
    return out


def launches(path):
    d = read_long(path)
    tot = defaultdict(float)
    n = defaultdict(int)
    for (_, name), m in d.items():
        v, u = m["gpu__time_duration.sum"]
        us = float(v) * {"ns": 1e-3, "us": 1.0, "ms": 1e3}.get(u, 1e-3)
        tot[short(name)] += us
        n[short(name)] += 1
    total = sum(tot.values())
    print(f"{'kernel':46s} {'launches':>8s} {'total us':>10s} {'us/launch':>10s} {'share':>7s}")
    for k in sorted(tot, key=lambda k: -tot[k]):
        print(f"{k:46s} {n[k]:8d} {tot[k]:10.1f} {tot[k] / n[k]:10.2f} {100 * tot[k] / total:6.1f}%")
    print(f"{'all':46s} {sum(n.values()):8d} {total:10.1f}")


def metrics(path):
    for (i, name), m in read_long(path).items():
        print(f"{i:4d} {short(name):44s} " + "  ".join(f"{k.split('.')[0].replace('__', ' ')} {v} {u}" for k, (v, u) in m.items()))


def full(path):
    for name, m in read_wide(path):
        print(f"== {short(name)}")
        for k in FULL_KEYS:
            if k in m and m[k][0] != "":
                print(f"   {k:78s} {m[k][0]:>14s} {m[k][1]}")
        stalls = []
        for k, (v, _) in m.items():
            if k.startswith("smsp__average_warps_issue_stalled_") and k.endswith("_per_issue_active.ratio"):
                try:
                    stalls.append((float(v), k[len("smsp__average_warps_issue_stalled_"):-len("_per_issue_active.ratio")]))
                except ValueError:
                    pass
        stalls.sort(reverse=True)
        print("   warp stalls per issue: " + ", ".join(f"{n} {v:.2f}" for v, n in stalls[:6]))


def to_bytes(v, u):
    return int(round(float(v) * {"byte": 1, "Kbyte": 1e3, "Mbyte": 1e6, "Gbyte": 1e9}.get(u, 1)))


def traffic(path, workload, out):
    kernels = {}
    for name, m in read_wide(path):
        kind = kind_of(name)
        if kind == "other" or kind in kernels:
            continue
        kernels[kind] = {"kernel": short(name), "dram_bytes_read": to_bytes(*m["dram__bytes_read.sum"]),
                         "dram_bytes_write": to_bytes(*m["dram__bytes_write.sum"])}
    json.dump({"workload": workload, "csrc_hash": accounting.csrc_hash(), "kernels": kernels,
               "note": "ncu --set full, caches flushed before the launch, one launch per kernel"},
              open(out, "w"), indent=1)
    print(json.dumps(kernels))


if __name__ == "__main__":
    cmd = sys.argv[1]
    {"launches": launches, "metrics": metrics, "full": full, "traffic": traffic}[cmd](*sys.argv[2:])
