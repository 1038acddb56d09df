"""Machine-written record of a kernel's DRAM traffic, taken from an ncu capture.

`bench.py` reports `roofline.traffic` (DRAM bytes per launch) from this record instead of measuring
under a profiler: a number printed by a run under ncu is never a bench value, and ncu is not part of
a plain benchmark run.  The record names the kernel, the sources it was captured on (with their
SHA-256, which `bench.py` recomputes and compares, so a record of another build is not used) and the
ratio of DRAM bytes to algorithmic bytes over all captured launches.

Writing a record (after the same bench command has exited 0 without ncu):

    python bench.py --sweep 8,64 --steps 4 --warmup 3 --no-cpu-baseline --no-pairings --e2e-steps 0 > plain.json
    ncu --metrics dram__bytes_read.sum,dram__bytes_write.sum,gpu__time_duration.sum --clock-control none \
        -k regex:attn_tc_kernel --csv --log-file launches.csv python bench.py <same arguments>
    python -m paper_2604_11035_b200.profile_record --kernel attn_tc_kernel --csv launches.csv --bench-json plain.json
"""
from __future__ import annotations

import argparse
import csv
import datetime
import hashlib
import json
import os

HERE = os.path.dirname(os.path.abspath(__file__))
PROFILES = os.path.join(os.path.dirname(HERE), "profiles")
KERNEL_SOURCES = {"attn_tc_kernel": ["isd_attn_tc.cu", "isd_internal.cuh"]}


def source_hash(sources) -> str:
    h = hashlib.sha256()
    for name in sources:
        with open(os.path.join(HERE, "csrc", name), "rb") as f:
            h.update(f.read())
    return h.hexdigest()


def record_path(kernel: str) -> str:
    return os.path.join(PROFILES, f"{kernel}_traffic_record.txt")


def load(kernel: str):
    p = record_path(kernel)
    if not os.path.exists(p):
        return None
    with open(p) as f:
        return json.load(f)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--kernel", required=True)
    ap.add_argument("--csv", required=True, help="ncu --csv log with dram__bytes_read.sum / dram__bytes_write.sum per launch")
    ap.add_argument("--bench-json", required=True, help="JSON line of the same bench command run without ncu")
    ap.add_argument("--command", default="")
    a = ap.parse_args()
    rows = [r for r in csv.reader(open(a.csv)) if len(r) > 10]
    hdr = rows[0]
    rd = wr = t_ns = 0.0
    ids = set()
    for r in rows[1:]:
        rec = dict(zip(hdr, r))
        if a.kernel not in rec["Kernel Name"]:
            continue
        ids.add(rec["ID"])
        v = float(rec["Metric Value"].replace(",", ""))
        if rec["Metric Name"] == "dram__bytes_read.sum":
            rd += v * {"byte": 1, "Kbyte": 1e3, "Mbyte": 1e6, "Gbyte": 1e9}[rec["Metric Unit"]]
        elif rec["Metric Name"] == "dram__bytes_write.sum":
            wr += v * {"byte": 1, "Kbyte": 1e3, "Mbyte": 1e6, "Gbyte": 1e9}[rec["Metric Unit"]]
        elif rec["Metric Name"] == "gpu__time_duration.sum":
            t_ns += v * {"ns": 1, "us": 1e3, "ms": 1e6, "nsecond": 1, "usecond": 1e3, "msecond": 1e6}[rec["Metric Unit"]]
    line = json.loads([l for l in open(a.bench_json) if l.startswith("{")][-1])
    alg, n = line["attn_bytes_all_launches"], line["attn_launches_all"]
    assert n == len(ids), f"the capture holds {len(ids)} launches of {a.kernel}, the plain run made {n}"
    sources = KERNEL_SOURCES[a.kernel]
    out = {"kernel": a.kernel, "sources": sources, "source_sha256": source_hash(sources),
           "workload": line["config"]["workload"], "command": a.command, "launches": n,
           "dram_bytes_read": rd, "dram_bytes_write": wr, "algorithmic_bytes": alg,
           "dram_bytes_per_algorithmic_byte": (rd + wr) / alg, "gpu_time_ns_under_ncu": t_ns,
           "captured": datetime.date.today().isoformat()}
    os.makedirs(PROFILES, exist_ok=True)
    with open(record_path(a.kernel), "w") as f:
        json.dump(out, f, indent=1)
        f.write("\n")
    print(json.dumps(out))


if __name__ == "__main__":
    main()
