"""Rewrites profiles/traffic.json from ncu captures of the three kernels.

    python -m paper_2305_19982_b200.traffic_table <dir with prof_fold / prof_apply / prof_wgrad .ncu-rep>

The captures are those of the commands given in profiles/*_67M.txt and
profiles/wgrad_fold_kernel_2cta_ldst_4096x4096_T4096.txt (fold and apply at 67,108,864
parameters, the fused call on 4096 x 4096 with 4096 tokens).  Per kernel the table keeps
dram__bytes_read.sum + dram__bytes_write.sum of the first captured launch, scaled for fold
and apply to the benchmark's 335,000,000-parameter launch (their traffic is proportional to
the size), and a hash of the kernel's source files; bench.py drops an entry whose hash no
longer matches, so a changed kernel reports no traffic until it has been captured again.
"""
from __future__ import annotations

import csv
import hashlib
import json
import subprocess
import sys
from pathlib import Path

ROOT = Path(__file__).resolve().parent.parent
CAPTURED_PARAMS = 67_108_864
BENCH_PARAMS = 335_000_000
SOURCES = {
    "fold_bf16": ["paper_2305_19982_b200/csrc/fold_apply.cu", "paper_2305_19982_b200/csrc/adama_device.cuh",
                  "paper_2305_19982_b200/csrc/stream_access.cuh"],
    "apply": ["paper_2305_19982_b200/csrc/fold_apply.cu", "paper_2305_19982_b200/csrc/adama_device.cuh",
              "paper_2305_19982_b200/csrc/stream_access.cuh"],
    "wgrad_fold": ["paper_2305_19982_b200/csrc/wgrad_fold.cu"],
}
REPORTS = {"fold_bf16": "prof_fold.ncu-rep", "apply": "prof_apply.ncu-rep", "wgrad_fold": "prof_wgrad.ncu-rep"}
UNITS = {"byte": 1.0, "Kbyte": 1e3, "Mbyte": 1e6, "Gbyte": 1e9}


def dram_bytes_of_first_launch(report: Path) -> float:
    out = subprocess.run(["ncu", "-i", str(report), "--page", "raw", "--csv"], capture_output=True,
                         text=True, check=True).stdout
    rows = list(csv.reader(out.splitlines()))
    head, units, first = rows[0], rows[1], rows[2]
    total = 0.0
    for name in ("dram__bytes_read.sum", "dram__bytes_write.sum"):
        k = head.index(name)
        total += float(first[k]) * UNITS[units[k]]
    return total


def source_hash(files) -> str:
    h = hashlib.sha256()
    for f in files:
        h.update((ROOT / f).read_bytes())
    return h.hexdigest()


def main(argv) -> int:
    if len(argv) != 2:
        print(__doc__)
        return 2
    folder = Path(argv[1])
    path = ROOT / "profiles" / "traffic.json"
    table = json.loads(path.read_text()) if path.exists() else {}
    for key, rep in REPORTS.items():
        b = dram_bytes_of_first_launch(folder / rep)
        entry = {"sources": SOURCES[key], "sha256": source_hash(SOURCES[key])}
        if key == "wgrad_fold":
            entry["bytes_per_launch"] = int(b)
        else:
            entry["bytes_per_launch"] = int(b * BENCH_PARAMS / CAPTURED_PARAMS)
            entry["bytes_per_param"] = round(b / CAPTURED_PARAMS, 1)
        table[key] = entry
        print(key, entry["bytes_per_launch"])
    path.write_text(json.dumps(table, indent=1) + "\n")
    return 0


if __name__ == "__main__":
    sys.exit(main(sys.argv))
