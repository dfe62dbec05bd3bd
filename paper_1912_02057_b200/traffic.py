"""Records the DRAM traffic of a workload's dominant kernel, as counted by Nsight Compute, in the tracked file
``profiles/traffic.json`` that ``bench.py`` reads for ``roofline.traffic``.

    python -m paper_1912_02057_b200.traffic --csv launches.csv --key WORKLOAD --kernel REGEX \\
        --sources paper_1912_02057_b200/csrc/rtn_conv_i8.cu ... [--launches-per-step N] [--skip N] --command "..."

The CSV is the log of

    ncu --metrics dram__bytes_read.sum,dram__bytes_write.sum --clock-control none --cache-control none \\
        -k regex:REGEX -s <warm-up launches> -c <several> --csv --log-file launches.csv \\
        python bench.py --workload WORKLOAD --eager --steps 4 --warmup 3 --no-cpu-baseline

over several CONSECUTIVE launches of the kernel on the benchmark's rotating buffers, WITHOUT the profiler's cache
flush between launches (--cache-control none): a kernel's fp32 output is still in L2 when it ends, so one launch
alone (or every launch, when the caches are flushed outside the counted window) shows almost no writes; with
the caches left alone the write-back of one launch falls into the window of the next ones, and the total
divided by the launches is the traffic of a launch (both counters come from one pass).  The record keeps a SHA-256 of every source file the kernel is built from; ``bench.py``
prints ``traffic: null`` once one of them has changed since the capture.
"""
import argparse
import csv
import hashlib
import json
import os
import re

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
TRAFFIC_FILE = os.path.join(ROOT, "profiles", "traffic.json")
UNIT = {"byte": 1.0, "Kbyte": 1e3, "Mbyte": 1e6, "Gbyte": 1e9}


def read_counters(path, kernel_regex, skip=0):
    """Sum of dram__bytes_read.sum and dram__bytes_write.sum over the launches (after the first `skip`) whose kernel
    name matches, and the number of such launches."""
    rows = []
    with open(path, newline="") as f:
        lines = [ln for ln in f if ln.startswith('"')]
    for row in csv.DictReader(lines):
        rows.append(row)
    pat = re.compile(kernel_regex)
    ids = []
    for r in rows:
        if pat.search(r["Kernel Name"]) and r["ID"] not in ids:
            ids.append(r["ID"])
    ids = ids[skip:]
    read = write = 0.0
    for r in rows:
        if r["ID"] not in ids:
            continue
        v = float(r["Metric Value"].replace(",", "")) * UNIT[r["Metric Unit"]]
        if r["Metric Name"] == "dram__bytes_read.sum":
            read += v
        elif r["Metric Name"] == "dram__bytes_write.sum":
            write += v
    return read, write, len(ids)


def sha256(path):
    h = hashlib.sha256()
    with open(path, "rb") as f:
        h.update(f.read())
    return h.hexdigest()


def main():
    ap = argparse.ArgumentParser(description=__doc__, formatter_class=argparse.RawDescriptionHelpFormatter)
    ap.add_argument("--csv", required=True)
    ap.add_argument("--key", required=True, help="workload name as bench.py prints it (plus /packed or /popc)")
    ap.add_argument("--kernel", required=True, help="regular expression on the kernel name")
    ap.add_argument("--sources", nargs="+", required=True, help="source files of the kernel, relative to the repository")
    ap.add_argument("--launches-per-step", type=int, default=1, help="matching launches that make up one step")
    ap.add_argument("--skip", type=int, default=0, help="matching launches to leave out at the start")
    ap.add_argument("--command", required=True, help="the command that was profiled")
    a = ap.parse_args()
    read, write, n = read_counters(a.csv, a.kernel, a.skip)
    if n == 0 or n % a.launches_per_step:
        raise SystemExit(f"{n} matching launches do not make whole steps of {a.launches_per_step}")
    steps = n // a.launches_per_step
    try:
        with open(TRAFFIC_FILE) as f:
            table = json.load(f)
    except (OSError, ValueError):
        table = {}
    table[a.key] = {
        "kernel": a.kernel, "bytes_per_launch": int(round((read + write) / steps)),
        "read_bytes_per_launch": int(round(read / steps)), "write_bytes_per_launch": int(round(write / steps)),
        "launches_captured": n, "launches_per_step": a.launches_per_step, "command": a.command,
        "sources": {rel: sha256(os.path.join(ROOT, rel)) for rel in a.sources},
    }
    with open(TRAFFIC_FILE, "w") as f:
        json.dump(table, f, indent=1, sort_keys=True)
        f.write("\n")
    print(json.dumps(table[a.key], indent=1))


if __name__ == "__main__":
    main()
