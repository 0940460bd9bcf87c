"""Turn an Nsight Compute launch list of `bench.py` into the short summaries kept under profiles/.

    python -m paper_2109_00170_b200.ncu_summary LAUNCHES.csv BENCH.json --out-md OUT.md [--out-traffic OUT.json]

LAUNCHES.csv is the `--csv --log-file` output of

    ncu --metrics gpu__time_duration.sum,dram__bytes_read.sum,dram__bytes_write.sum \\
        --clock-control none --nvtx --nvtx-include "alcs_timed/" --csv --log-file LAUNCHES.csv \\
        python bench.py --steps 2 --warmup 3 --no-cpu-baseline --e2e-steps 0 --no-batch1

and BENCH.json is the JSON line the same command printed when run without ncu.  The launches inside
the "alcs_timed" range are the layers of the stack in order, repeated `steps` times, so convolution launch i
is layer i mod n_layers (a row-repacking launch belongs to the convolution after it).  Per-launch times under ncu are cold-cache and serialised: the SHARES are what
can be compared with the live CUDA-event timings, not the absolutes.
"""
from __future__ import annotations

import argparse
import csv
import json
import os
import re
import sys
from collections import OrderedDict, defaultdict


def read_launches(path):
    """[(kernel name, {metric: value})] in launch order, from ncu's long-format CSV log."""
    rows = []
    with open(path, newline="") as f:
        lines = [l for l in f if not l.startswith("==")]
    rd = csv.DictReader(lines)
    by_id = OrderedDict()
    for r in rd:
        if "ID" not in r or r.get("Metric Name") is None:
            continue
        k = by_id.setdefault(r["ID"], {"name": r["Kernel Name"], "m": {}})
        val = r["Metric Value"].replace(",", "")
        try:
            v = float(val)
        except ValueError:
            continue
        unit = (r.get("Metric Unit") or "").lower()
        scale = {"ns": 1e-3, "us": 1.0, "usecond": 1.0, "nsecond": 1e-3, "ms": 1e3, "msecond": 1e3, "second": 1e6,
                 "byte": 1.0, "kbyte": 1e3, "mbyte": 1e6, "gbyte": 1e9}.get(unit, 1.0)
        k["m"][r["Metric Name"]] = v * scale
    for k in by_id.values():
        rows.append((k["name"], k["m"]))
    return rows


def source_hash():
    import hashlib
    h = hashlib.sha256()
    d = os.path.join(os.path.dirname(os.path.abspath(__file__)), "csrc")
    for f in sorted(os.listdir(d)):
        if f.startswith(("alcs_conv2d", "alcs_project")):
            continue        # other entry points: they do not change the pointwise kernels
        h.update(open(os.path.join(d, f), "rb").read())
    return h.hexdigest()[:16]


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("launches")
    ap.add_argument("bench_json")
    ap.add_argument("--out-md", required=True)
    ap.add_argument("--out-traffic")
    ap.add_argument("--command", default="")
    a = ap.parse_args()

    launches = read_launches(a.launches)
    bench = None
    for line in open(a.bench_json):
        line = line.strip()
        if line.startswith("{"):
            bench = json.loads(line)
    if bench is None:
        sys.exit("no JSON line in " + a.bench_json)
    layers = bench["layers"]
    nl = len(layers)
    # A layer whose X rows are not a multiple of 16 bytes launches the row-repacking kernel first;
    # that launch is counted with the convolution that follows it.
    n_conv = sum(1 for name, _ in launches if "spconv1x1_" in name)
    if not n_conv or n_conv % nl:
        sys.exit(f"{n_conv} convolution launches do not divide into {nl} layers")
    reps = n_conv // nl

    per_kernel = defaultdict(lambda: [0, 0.0])
    per_layer = [dict(t=0.0, rd=0.0, wr=0.0) for _ in range(nl)]
    total = 0.0
    i = 0
    for name, m in launches:
        t = m.get("gpu__time_duration.sum", 0.0)
        short = re.sub(r"^void\s+|alcs::|\(.*\)$", "", name)
        per_kernel[short][0] += 1
        per_kernel[short][1] += t
        L = per_layer[i % nl]
        if "spconv1x1_" in name:
            i += 1
        L["t"] += t / reps
        L["rd"] += m.get("dram__bytes_read.sum", 0.0) / reps
        L["wr"] += m.get("dram__bytes_write.sum", 0.0) / reps
        total += t

    live_total = sum(r["us"] for r in layers)
    out = []
    out.append(f"# ncu launch list: {bench['config']['workload']} ({nl} layers x {reps} steps)\n")
    if a.command:
        out.append("Command (run once without ncu first, then under ncu):\n\n    " + a.command + "\n")
    out.append("Per-launch times under ncu are cold-cache and serialised; compare the SHARE column with "
               "the live share (CUDA events inside bench.py), not the absolute times.\n")
    out.append("## Per kernel variant\n")
    out.append("| kernel | launches | total us | share |")
    out.append("|---|---|---|---|")
    for k, (n, t) in sorted(per_kernel.items(), key=lambda kv: -kv[1][1]):
        out.append(f"| `{k}` | {n} | {t:.1f} | {100 * t / total:.1f} % |")
    out.append("\n## Per layer (mean over the captured steps)\n")
    out.append("| layer | ncu us | ncu share | live us | live share | algorithmic MB | DRAM read MB | DRAM write MB | DRAM / algorithmic |")
    out.append("|---|---|---|---|---|---|---|---|---|")
    traffic = {}
    for L, r in zip(per_layer, layers):
        dram = L["rd"] + L["wr"]
        out.append(f"| {r['layer']} | {L['t']:.1f} | {100 * L['t'] * reps / total:.1f} % | {r['us']:.1f} | "
                   f"{100 * r['us'] / live_total:.1f} % | {r['mbytes']:.1f} | {L['rd'] / 1e6:.1f} | {L['wr'] / 1e6:.1f} | "
                   f"{dram / 1e6 / r['mbytes']:.2f} |")
        traffic[r["layer"]] = {"dram_bytes": round(dram), "cfg": r["cfg"]}
    out.append("")
    out.append("DRAM write bytes are below the size of Y where Y (or its tail) is still dirty in the 126 MB L2 "
               "when the kernel ends; DRAM read bytes equal the size of X, i.e. X is fetched from HBM once "
               "even where several row groups stream the same tile (the repeats hit in L2).")
    out.append("")
    with open(a.out_md, "w") as f:
        f.write("\n".join(out))
    if a.out_traffic:
        with open(a.out_traffic, "w") as f:
            json.dump({"source_hash": source_hash(), "note": "dram__bytes_read.sum + dram__bytes_write.sum per launch, "
                       "from the ncu launch list summarised in " + os.path.basename(a.out_md), "layers": traffic}, f, indent=1)


if __name__ == "__main__":
    main()
