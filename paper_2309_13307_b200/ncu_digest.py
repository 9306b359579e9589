"""Turns Nsight Compute CSV logs of the round kernels into the short summaries kept under profiles/.

    python -m paper_2309_13307_b200.ncu_digest launches  <ncu --csv log>  <out.md>   "<command that made the log>"
    python -m paper_2309_13307_b200.ncu_digest dram      <ncu --csv log>  <out.json> --d D --ms M1,M2,...

`launches`: per kernel its launch count, total device time and share (from gpu__time_duration.sum).
`dram`: per (kernel, m) the DRAM bytes of one launch (dram__bytes_read.sum + dram__bytes_write.sum), stamped with
the digest of the CUDA sources so that bench.py can tell whether the counters still describe the code.  The log
must come from `bench.py --d D --m M1 M2 ...`, which launches each kernel once per m, in that order, per step.
"""
from __future__ import annotations

import csv
import glob
import hashlib
import json
import os
import re
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


# The files project_kernel and reconstruct_kernel (the two kernels the DRAM capture covers) are compiled from.
ROUND_KERNEL_SOURCES = ("core_internal.h", "core_project.cu", "core_reconstruct.cu", "core_rng.cuh")


def csrc_digest() -> str:
    """Digest of the sources of the two captured kernels: the stored counters describe exactly this code."""
    h = hashlib.sha256()
    for name in ROUND_KERNEL_SOURCES:
        h.update(name.encode())
        h.update(open(os.path.join(ROOT, "paper_2309_13307_b200", "csrc", name), "rb").read())
    return h.hexdigest()


def read_long_csv(path: str):
    """Rows of an `ncu --csv --log-file` log as dicts (skips the ==PROF== chatter)."""
    lines = [l for l in open(path, newline="") if l.startswith('"')]
    return list(csv.DictReader(lines))


def to_number(text: str) -> float:
    return float(text.replace(",", ""))


def short_name(kernel: str) -> str:
    m = re.search(r"(\w+_kernel)", kernel)
    return m.group(1) if m else kernel[:40]


def to_bytes(value: float, unit: str) -> float:
    scale = {"byte": 1, "Kbyte": 1e3, "Mbyte": 1e6, "Gbyte": 1e9, "Tbyte": 1e12}
    return value * scale[unit]


def to_ms(value: float, unit: str) -> float:
    scale = {"ns": 1e-6, "us": 1e-3, "ms": 1.0, "s": 1e3, "nsecond": 1e-6, "usecond": 1e-3, "msecond": 1.0, "second": 1e3}
    return value * scale[unit]


def launches(log: str, out: str, command: str) -> None:
    per = {}
    for r in read_long_csv(log):
        if r["Metric Name"] != "gpu__time_duration.sum":
            continue
        k = short_name(r["Kernel Name"])
        e = per.setdefault(k, [0, 0.0])
        e[0] += 1
        e[1] += to_ms(to_number(r["Metric Value"]), r["Metric Unit"])
    total = sum(v[1] for v in per.values())
    with open(out, "w") as f:
        f.write("# Launch list of the round kernels (ncu, gpu__time_duration.sum, one pass)\n\n")
        f.write(f"Command: `{command}`\n\n")
        f.write("Per-launch times under the profiler are serialised and cold-cache: compare shares, not absolutes.\n\n")
        f.write("| kernel | launches | total ms | share |\n|---|---|---|---|\n")
        for k, (cnt, ms) in sorted(per.items(), key=lambda kv: -kv[1][1]):
            f.write(f"| {k} | {cnt} | {ms:.3f} | {100 * ms / total:.2f} % |\n")


def dram(log: str, out: str, d: int, ms) -> None:
    rows = read_long_csv(log)
    by_id = {}
    for r in rows:
        e = by_id.setdefault(r["ID"], {"kernel": short_name(r["Kernel Name"]), "grid": r.get("Grid Size", "")})
        if r["Metric Name"].startswith("dram__bytes"):
            e[r["Metric Name"]] = to_bytes(to_number(r["Metric Value"]), r["Metric Unit"])
        if r["Metric Name"] == "gpu__time_duration.sum":
            e["ms"] = to_ms(to_number(r["Metric Value"]), r["Metric Unit"])
    caps = []
    seen = {}
    for _, e in sorted(by_id.items(), key=lambda kv: int(kv[0])):
        if "dram__bytes_read.sum" not in e:
            continue
        idx = seen.get(e["kernel"], 0)
        seen[e["kernel"]] = idx + 1
        caps.append({"kernel": e["kernel"].replace("_kernel", ""), "m": ms[idx % len(ms)], "grid": e["grid"], "d": d,
                     "ms_under_ncu": e.get("ms"),
                     "dram_read": e["dram__bytes_read.sum"], "dram_write": e["dram__bytes_write.sum"],
                     "dram_bytes": e["dram__bytes_read.sum"] + e["dram__bytes_write.sum"]})
    json.dump({"csrc_sha256": csrc_digest(), "captures": caps}, open(out, "w"), indent=1)


def main(argv):
    if len(argv) >= 5 and argv[1] == "launches":
        launches(argv[2], argv[3], argv[4])
    elif len(argv) >= 8 and argv[1] == "dram" and argv[4] == "--d" and argv[6] == "--ms":
        dram(argv[2], argv[3], int(argv[5]), [int(x) for x in argv[7].split(",")])
    else:
        sys.stderr.write(__doc__)
        return 2
    return 0


if __name__ == "__main__":
    sys.exit(main(sys.argv))
