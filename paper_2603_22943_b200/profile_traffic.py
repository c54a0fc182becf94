"""Records the DRAM traffic of a kernel from an ncu capture, for the benchmark's roofline line.

``python -m paper_2603_22943_b200.profile_traffic <raw.csv> <kernel regex> <record name> <kernel source file>``
reads the CSV of ``ncu -i <report> --page raw --csv``, averages ``dram__bytes_read.sum + dram__bytes_write.sum`` over the
captured launches whose kernel name matches, and stores the figure in ``profiles/dram_traffic.json`` together with the
hash of the kernel's source file, so that the benchmark stops quoting it once the kernel has changed.
"""
from __future__ import annotations

import csv
import hashlib
import json
import os
import re
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
UNIT = {"byte": 1.0, "Kbyte": 1e3, "Mbyte": 1e6, "Gbyte": 1e9}


def dram_bytes_per_launch(csv_path: str, kernel_regex: str):
    """Accepts both CSV forms ncu writes: the raw page of a report (one row per launch, one column per metric) and the
    log of a ``--metrics ... --csv`` run (one row per launch and metric)."""
    rows = [r for r in csv.reader(open(csv_path)) if len(r) > 5]
    hdr = next(r for r in rows if "Kernel Name" in r)
    col = {h: i for i, h in enumerate(hdr)}
    data = rows[rows.index(hdr) + 1:]
    per_launch = {}
    if "Metric Name" in col:
        for r in data:
            if r[col["Metric Name"]] in ("dram__bytes_read.sum", "dram__bytes_write.sum") and re.search(kernel_regex, r[col["Kernel Name"]]):
                v = float(r[col["Metric Value"]].replace(",", "")) * UNIT[r[col["Metric Unit"]]]
                per_launch[r[col["ID"]]] = per_launch.get(r[col["ID"]], 0.0) + v
    else:
        units = data[0]
        rd, wr = col["dram__bytes_read.sum"], col["dram__bytes_write.sum"]
        for r in data[1:]:
            if re.search(kernel_regex, r[col["Kernel Name"]]):
                per_launch[r[col["ID"]]] = float(r[rd]) * UNIT[units[rd]] + float(r[wr]) * UNIT[units[wr]]
    vals = list(per_launch.values())
    if not vals:
        raise SystemExit(f"no launch matches {kernel_regex!r}")
    return sum(vals) / len(vals), len(vals)


def main(argv):
    csv_path, regex, name, source = argv
    per_launch, n = dram_bytes_per_launch(csv_path, regex)
    path = os.path.join(ROOT, "profiles", "dram_traffic.json")
    rec = json.load(open(path)) if os.path.exists(path) else {}
    src = os.path.join(ROOT, source)
    rec[name] = {"dram_bytes_per_launch": int(round(per_launch)), "launches_averaged": n, "source": source,
                 "source_sha256": hashlib.sha256(open(src, "rb").read()).hexdigest()}
    json.dump(rec, open(path, "w"), indent=1, sort_keys=True)
    print(f"{name}: {per_launch / 1e6:.3f} MB per launch over {n} launches -> {path}")


if __name__ == "__main__":
    main(sys.argv[1:])
