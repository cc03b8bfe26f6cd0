#!/usr/bin/env python
"""Turns one ncu capture of bench.py's patch-coder launches into profiles/patch_coder_dram_traffic.json.

Capture (one B200, one pass per launch, after the same bench command has run without ncu):

    python bench.py --steps 1 --warmup 3 --no-e2e --no-wbin --no-cpu-baseline
    ncu --metrics dram__bytes_read.sum,dram__bytes_write.sum --clock-control none -k regex:"pixhist|patches" \\
        -s <launches of the warm-up steps> -c <launches of one step> --csv --log-file traffic.csv \\
        python bench.py --steps 1 --warmup 3 --no-e2e --no-wbin --no-cpu-baseline
    python record_traffic.py traffic.csv

The launches of one step are attributed to the 16 layers in order (each layer's coder launches one main kernel
and the kernels that take what it marked).  The record carries a hash of the coder's sources; bench.py quotes it
only while that hash matches.
"""
import csv
import json
import sys

import bench
from dab_synth import configs


def main():
    path = sys.argv[1]
    rows = list(csv.DictReader(line for line in open(path, errors="replace") if line.startswith('"')))
    per_launch = {}
    for r in rows:
        d = per_launch.setdefault(int(r["ID"]), {"name": r["Kernel Name"], "bytes": 0.0})
        if r["Metric Name"] in ("dram__bytes_read.sum", "dram__bytes_write.sum"):
            v = float(r["Metric Value"].replace(",", ""))
            unit = r["Metric Unit"].lower()
            d["bytes"] += v * {"byte": 1.0, "kbyte": 1e3, "mbyte": 1e6, "gbyte": 1e9}[unit]
    launches = [per_launch[k] for k in sorted(per_launch)]
    layers = configs.config5(256)
    out, i = {}, 0
    for L in layers:
        n = bench.patch_launches(L, "auto")
        out[L.name] = sum(x["bytes"] for x in launches[i:i + n])
        i += n
    if i != len(launches):
        raise SystemExit("captured %d launches, one step has %d" % (len(launches), i))
    rec = {"source_sha256": bench.patch_coder_source_hash(), "batch": 256, "dense": False,
           "command": "ncu --metrics dram__bytes_read.sum,dram__bytes_write.sum --clock-control none -k regex:pixhist|patches "
                      "python bench.py --steps 1 --warmup 3 --no-e2e --no-wbin --no-cpu-baseline (the timed step's launches)",
           "dram_bytes_per_launch": out}
    with open(bench.TRAFFIC_RECORD, "w") as f:
        json.dump(rec, f, indent=1)
    alg = {L.name: 4 * L.N * L.C * L.H * L.W + L.patches * (4 * ((L.n + 31) // 32) + 12) for L in layers}
    for L in layers:
        print("%s measured %.1f MB algorithmic %.1f MB ratio %.3f" % (L.name, out[L.name] / 1e6, alg[L.name] / 1e6, out[L.name] / alg[L.name]))


if __name__ == "__main__":
    main()
