"""Records the DRAM traffic of one guide_simulate call from a profiler capture, for bench.py's
`roofline.traffic`.

  ncu -i capture.ncu-rep --page raw --csv > capture.csv
  python -m paper_2412_04788_b200.traffic_record capture.csv 16777216 [launches per call = 2]

sums dram__bytes_read.sum + dram__bytes_write.sum over the closed-form kernels' launches of one call
and writes profiles/k_closed_form_c5_traffic.json together with a hash of the kernel sources, so
that the figure is dropped (reported as null) once those sources change.
"""
from __future__ import annotations

import csv
import hashlib
import json
import os
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
SOURCES = ("closed_form.cu", "line_walk.cuh", "model_walk.cuh", "model.cuh", "tiled.cuh")
OUT = os.path.join(HERE, "..", "profiles", "k_closed_form_c5_traffic.json")
UNIT = {"byte": 1.0, "Kbyte": 1e3, "Mbyte": 1e6, "Gbyte": 1e9}


def sources_sha256() -> str:
    h = hashlib.sha256()
    for name in SOURCES:
        with open(os.path.join(HERE, "csrc", name), "rb") as f:
            h.update(f.read())
    return h.hexdigest()


def main(argv):
    path, n_configs = argv[1], int(argv[2])
    per_call = int(argv[3]) if len(argv) > 3 else 2
    rows = list(csv.reader(open(path)))
    hdr, units, body = rows[0], rows[1], rows[2:]
    name_col = hdr.index("Kernel Name")
    cols = [hdr.index("dram__bytes_read.sum"), hdr.index("dram__bytes_write.sum")]
    launches = [r for r in body if "k_closed_form" in r[name_col]]
    if len(launches) < per_call:
        raise SystemExit("the capture holds fewer closed-form launches than one call makes")
    total = 0.0
    for r in launches[-per_call:]:                       # the last call captured
        for c in cols:
            total += float(r[c].replace(",", "")) * UNIT[units[c]]
    rec = {"configs": n_configs, "dram_bytes_per_call": int(total), "launches_per_call": per_call,
           "kernels": [r[name_col].split("(")[0] for r in launches[-per_call:]], "sources_sha256": sources_sha256(),
           "capture": os.path.basename(path)}
    with open(OUT, "w") as f:
        json.dump(rec, f, indent=1)
    print(json.dumps(rec))


if __name__ == "__main__":
    main(sys.argv)
