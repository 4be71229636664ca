"""DRAM traffic per kernel launch, recorded from an ncu capture and tied to the kernel's source.

    python -m paper_2603_14303_b200.ncu_traffic <ncu.csv> --kernel decode_mma_kernel \
        --stage decode --workload cfg1-llama3-8b-32k [--scale 1.0] [--note "..."]

reads a CSV written by ``ncu --csv --page raw`` (or ``ncu --csv --metrics dram__bytes_read.sum,
dram__bytes_write.sum``), averages ``dram__bytes_read.sum + dram__bytes_write.sum`` over the captured
launches of the named kernel and stores the figure in ``profiles/traffic.txt`` (JSON) together with a hash
of the kernel's source file.  ``lookup`` returns the figure only while that file is unchanged, so a
benchmark line never quotes counters of a kernel that no longer exists.
"""
from __future__ import annotations

import argparse
import csv
import hashlib
import json
import os

HERE = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(HERE)
RECORD = os.path.join(ROOT, "profiles", "traffic.txt")

# stage -> source file whose change invalidates the record
SOURCES = {"decode": "csrc/decode_mma.cu", "compress": "csrc/compress_fused.cu", "compress_layers": "csrc/compress_fused.cu",
           "prefill": "csrc/prefill_umma.cu"}

_UNITS = {"byte": 1.0, "Kbyte": 1e3, "Mbyte": 1e6, "Gbyte": 1e9, "Tbyte": 1e12}


def source_hash(stage: str) -> str | None:
    path = os.path.join(HERE, SOURCES[stage])
    if not os.path.exists(path):
        return None
    with open(path, "rb") as f:
        return hashlib.sha256(f.read()).hexdigest()[:16]


def lookup(workload: str, stage: str):
    """Recorded DRAM bytes per launch for (workload, stage), or None if absent or stale."""
    if not os.path.exists(RECORD):
        return None
    with open(RECORD) as f:
        rec = json.load(f)
    e = rec.get(f"{workload}/{stage}")
    if not e or e.get("source_sha256_16") != source_hash(stage):
        return None
    return float(e["dram_bytes_per_launch"])


def parse_ncu_csv(path: str, kernel: str):
    """Per-launch (read, write) byte totals of launches whose name contains ``kernel``.

    Takes both layouts ncu writes: the raw page (one row per launch, one column per metric, a units
    row under the header) and the long form (one row per launch and metric)."""
    with open(path, newline="") as f:
        rows = [r for r in csv.reader(f) if r]
    start = next(i for i, r in enumerate(rows) if "Kernel Name" in r)
    head, body = rows[start], rows[start + 1:]
    name_col = head.index("Kernel Name")
    out = []
    if "Metric Name" in head:   # long form
        mcol, vcol, ucol, idcol = head.index("Metric Name"), head.index("Metric Value"), head.index("Metric Unit"), head.index("ID")
        per = {}
        for r in body:
            if kernel not in r[name_col] or r[mcol] not in ("dram__bytes_read.sum", "dram__bytes_write.sum"):
                continue
            per.setdefault(r[idcol], {})[r[mcol]] = float(r[vcol].replace(",", "")) * _UNITS.get(r[ucol], 1.0)
        for v in per.values():
            out.append((v.get("dram__bytes_read.sum", 0.0), v.get("dram__bytes_write.sum", 0.0)))
    else:                       # raw page: first body row holds the units
        units, body = body[0], body[1:]
        rc, wc = head.index("dram__bytes_read.sum"), head.index("dram__bytes_write.sum")
        for r in body:
            if kernel in r[name_col]:
                out.append((float(r[rc].replace(",", "")) * _UNITS.get(units[rc], 1.0),
                            float(r[wc].replace(",", "")) * _UNITS.get(units[wc], 1.0)))
    return out


def main():
    ap = argparse.ArgumentParser(description=__doc__, formatter_class=argparse.RawDescriptionHelpFormatter)
    ap.add_argument("csv")
    ap.add_argument("--kernel", required=True)
    ap.add_argument("--stage", required=True, choices=sorted(SOURCES))
    ap.add_argument("--workload", required=True)
    ap.add_argument("--scale", type=float, default=1.0,
                    help="units of a full launch / units of the captured launch, when a smaller case was captured")
    ap.add_argument("--note", default="")
    a = ap.parse_args()
    launches = parse_ncu_csv(a.csv, a.kernel)
    if not launches:
        raise SystemExit(f"no launch of {a.kernel} in {a.csv}")
    rd = sum(x for x, _ in launches) / len(launches) * a.scale
    wr = sum(y for _, y in launches) / len(launches) * a.scale
    rec = {}
    if os.path.exists(RECORD):
        with open(RECORD) as f:
            rec = json.load(f)
    rec[f"{a.workload}/{a.stage}"] = {
        "kernel": a.kernel, "launches_captured": len(launches), "dram_read_bytes_per_launch": rd,
        "dram_write_bytes_per_launch": wr, "dram_bytes_per_launch": rd + wr, "scale": a.scale,
        "source": SOURCES[a.stage], "source_sha256_16": source_hash(a.stage), "note": a.note}
    os.makedirs(os.path.dirname(RECORD), exist_ok=True)
    with open(RECORD, "w") as f:
        json.dump(rec, f, indent=1, sort_keys=True)
        f.write("\n")
    print(json.dumps(rec[f"{a.workload}/{a.stage}"]))


if __name__ == "__main__":
    main()
