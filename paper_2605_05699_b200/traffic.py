"""Records the DRAM traffic of one captured launch for bench.py's `roofline.traffic`.

    ncu -i capture.ncu-rep --page raw --csv > capture.csv        (or the --csv --log-file of a --metrics capture)
    python -m paper_2605_05699_b200.traffic capture.csv decode kvq_umma_decode.cu

Reads dram__bytes_read.sum and dram__bytes_write.sum of the first kernel row of an ncu CSV and stores them, with a hash of
the kernel's source file, in profiles/dram_traffic.json.  bench.py reports the sum while that source file is unchanged and
null afterwards: counters of a kernel that has since changed are not quoted.
"""
from __future__ import annotations

import csv
import hashlib
import json
import os
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
UNITS = {"byte": 1.0, "Kbyte": 1e3, "Mbyte": 1e6, "Gbyte": 1e9}


def _read(path: str):
    rows = [r for r in csv.reader(open(path)) if r and not r[0].startswith("==")]
    hdr = rows[0]
    if "Metric Name" in hdr:                       # long form: one metric per row
        i_n, i_u, i_v = hdr.index("Metric Name"), hdr.index("Metric Unit"), hdr.index("Metric Value")
        out = {}
        for r in rows[1:]:
            if r[i_n] in ("dram__bytes_read.sum", "dram__bytes_write.sum") and r[i_n] not in out:
                out[r[i_n]] = float(r[i_v].replace(",", "")) * UNITS[r[i_u]]
        return out
    units, vals = rows[1], rows[2]                 # raw page: one column per metric, a units row, then kernels
    return {k: float(vals[hdr.index(k)].replace(",", "")) * UNITS[units[hdr.index(k)]]
            for k in ("dram__bytes_read.sum", "dram__bytes_write.sum")}


def main():
    if len(sys.argv) != 4:
        raise SystemExit(__doc__)
    path, which, source = sys.argv[1:]
    m = _read(path)
    with open(os.path.join(ROOT, "paper_2605_05699_b200", "csrc", source), "rb") as f:
        sha = hashlib.sha256(f.read()).hexdigest()[:16]
    out = os.path.join(ROOT, "profiles", "dram_traffic.json")
    rec = json.load(open(out)) if os.path.exists(out) else {}
    rec[which] = {"dram_bytes_read": int(m["dram__bytes_read.sum"]), "dram_bytes_write": int(m["dram__bytes_write.sum"]),
                  "source": source, "source_sha16": sha, "capture": os.path.basename(path)}
    with open(out, "w") as f:
        json.dump(rec, f, indent=1, sort_keys=True)
        f.write("\n")
    print(json.dumps(rec[which]))


if __name__ == "__main__":
    main()
