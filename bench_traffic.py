"""Writes profiles/dram_traffic.json from an ncu capture of bench.py's DRAM counters.

    python bench.py --steps 2 --warmup 3 --no-e2e --no-cpu-baseline --secondary "" --no-block-chain      # must exit 0 first
    ncu --metrics dram__bytes_read.sum,dram__bytes_write.sum --clock-control none -k regex:linear_tc_ \
        --csv --log-file dram_stack.csv \
        python bench.py --steps 2 --warmup 3 --no-e2e --no-cpu-baseline --secondary "" --no-block-chain
    python bench_traffic.py dram_stack.csv --workload deit_b_stack_b256

The two counters are one pass, so the full-size workload is captured directly.  Only the launches that carry several
layers (the launches of the timed steps) are counted: per kernel family, bytes read + written summed over those
launches and divided by the number of steps seen.  The record carries the SHA-256 of the kernel sources
(bench.kernel_source_hash); bench.py reports the traffic only while that hash matches the tree.
"""
from __future__ import annotations

import argparse
import collections
import csv
import json
import os
import re

import bench

COMMAND = ("ncu --metrics dram__bytes_read.sum,dram__bytes_write.sum --clock-control none -k regex:linear_tc_ --csv "
           "--log-file dram_stack.csv python bench.py --workload %s --steps 2 --warmup 3 --no-e2e --no-cpu-baseline "
           "--secondary \"\" --no-block-chain")


def family_bytes(csv_path):
    rows = list(csv.reader(line for line in open(csv_path) if line.startswith('"')))
    hdr = rows[0]
    kid, name, metric, value = (hdr.index(k) for k in ("ID", "Kernel Name", "Metric Name", "Metric Value"))
    launches = collections.OrderedDict()
    for r in rows[1:]:
        d = launches.setdefault(r[kid], {"name": r[name], "bytes": 0.0})
        if r[metric] in ("dram__bytes_read.sum", "dram__bytes_write.sum"):
            d["bytes"] += float(r[value].replace(",", ""))
    fam = collections.OrderedDict()
    for d in launches.values():
        m = re.search(r"(linear_tc_\w+?)_kernel<([^>]*)>", d["name"])
        if not m:
            continue
        args = [a.strip() for a in m.group(2).split(",")]
        # the layer-table launches are the instantiations whose layer capacity is above one: <bf16, capacity, ...> for
        # the sparse kernels, <bf16, form, capacity> for the dense pair kernel
        capacity = int(args[2]) if m.group(1) == "linear_tc_pair" else int(args[1])
        if capacity <= 1:
            continue
        f = fam.setdefault(m.group(1), {"bytes": 0.0, "launches": 0})
        f["bytes"] += d["bytes"]
        f["launches"] += 1
    return fam


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("csv")
    ap.add_argument("--workload", default="deit_b_stack_b256")
    ap.add_argument("--out", default=os.path.join(bench.ROOT, "profiles", "dram_traffic.json"))
    args = ap.parse_args()
    fam = family_bytes(args.csv)
    steps = min(f["launches"] for f in fam.values())          # the families with one launch per step
    captures = []
    for name, f in fam.items():
        captures.append({"workload": args.workload, "kernel": name, "dram_bytes_per_step": f["bytes"] / steps,
                         "launches_per_step": f["launches"] / steps, "steps_captured": steps,
                         "csrc_sha256": bench.kernel_source_hash(), "command": COMMAND % args.workload})
    try:
        with open(args.out) as fh:
            old = [c for c in json.load(fh).get("captures", []) if c.get("workload") != args.workload]
    except (OSError, ValueError):
        old = []
    with open(args.out, "w") as fh:
        json.dump({"captures": old + captures}, fh, indent=1)
    for c in captures:
        print(c["kernel"], "%.3f GB per step, %g launches per step" % (c["dram_bytes_per_step"] / 1e9, c["launches_per_step"]))


if __name__ == "__main__":
    main()
