"""Record of the DRAM traffic of the dominant kernels, taken from a profiler capture.

    python -m paper_2608_28158_b200.traffic --csv <ncu raw csv> --kernel tc_bwd_kernel --units <units> \
        --workload cfg2 --out profiles/traffic.json

reads the `dram__bytes_read.sum` and `dram__bytes_write.sum` columns of an `ncu --csv --page raw` export (or of a
`--metrics dram__bytes_read.sum,dram__bytes_write.sum --csv` log), sums them over the captured launches of the named
kernel and stores bytes per unit (`--units` = the units, e.g. token-heads, those launches processed together) with the
git commit and a hash of the kernel's source files.  The benchmark reads the record back and reports `traffic` only
while that hash still matches the sources, so a number never outlives the kernel it was measured on."""
from __future__ import annotations

import argparse
import csv
import hashlib
import json
import os
import subprocess

HERE = os.path.dirname(os.path.abspath(__file__))
SOURCES = {"tc_bwd_kernel": ["csrc/la_tc_bwd.cu", "csrc/tc_common.cuh"],
           "tc_fwd_kernel": ["csrc/la_tc_fwd.cu", "csrc/tc_common.cuh"]}


def source_hash(files):
    h = hashlib.sha256()
    for f in files:
        path = os.path.join(HERE, f)
        if not os.path.exists(path):
            return None
        with open(path, "rb") as fh:
            h.update(fh.read())
    return h.hexdigest()


def load(path):
    if not os.path.exists(path):
        return {}
    with open(path) as f:
        return json.load(f)


def _to_bytes(value, unit):
    scale = {"byte": 1, "bytes": 1, "kbyte": 1e3, "mbyte": 1e6, "gbyte": 1e9, "tbyte": 1e12}
    return float(value.replace(",", "")) * scale.get(unit.strip().lower(), 1)


def dram_bytes(csv_path, kernel):
    """(total DRAM bytes, launches) of `kernel` in an ncu csv: the wide `--page raw` form (one row per launch, one
    column per metric, a units row under the header) or the long form (one row per launch and metric)."""
    with open(csv_path, newline="") as f:
        lines = [ln for ln in f if ln.startswith('"')]
    rows = list(csv.reader(lines))
    head = rows[0]
    total, launches = 0.0, set()
    if "Metric Name" in head:                                   # long form
        i_k, i_n, i_u, i_v, i_id = (head.index(c) for c in ("Kernel Name", "Metric Name", "Metric Unit", "Metric Value", "ID"))
        for r in rows[1:]:
            if kernel in r[i_k] and r[i_n] in ("dram__bytes_read.sum", "dram__bytes_write.sum"):
                total += _to_bytes(r[i_v], r[i_u])
                launches.add(r[i_id])
    else:                                                        # wide form: second row holds the units
        units = rows[1]
        i_k, i_id = head.index("Kernel Name"), head.index("ID")
        cols = [head.index(c) for c in ("dram__bytes_read.sum", "dram__bytes_write.sum")]
        for r in rows[2:]:
            if kernel in r[i_k]:
                total += sum(_to_bytes(r[c], units[c]) for c in cols)
                launches.add(r[i_id])
    return total, len(launches)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--csv", required=True)
    ap.add_argument("--kernel", required=True, choices=sorted(SOURCES))
    ap.add_argument("--units", type=float, required=True, help="units (token-heads) processed by the captured launches")
    ap.add_argument("--workload", required=True)
    ap.add_argument("--out", default=os.path.join(HERE, "..", "profiles", "traffic.json"))
    a = ap.parse_args()
    total, n = dram_bytes(a.csv, a.kernel)
    if not n:
        raise SystemExit(f"no launch of {a.kernel} in {a.csv}")
    try:
        commit = subprocess.check_output(["git", "-C", HERE, "rev-parse", "--short", "HEAD"], text=True).strip()
    except (OSError, subprocess.CalledProcessError):
        commit = "unknown"
    rec = load(a.out)
    rec[a.kernel] = {"dram_bytes_per_unit": total / a.units, "unit": "token-head", "launches": n, "workload": a.workload,
                     "commit": commit, "sources": SOURCES[a.kernel], "source_sha256": source_hash(SOURCES[a.kernel])}
    with open(a.out, "w") as f:
        json.dump(rec, f, indent=1)
        f.write("\n")
    print(json.dumps(rec[a.kernel]))


if __name__ == "__main__":
    main()
