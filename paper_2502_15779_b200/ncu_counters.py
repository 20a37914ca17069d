"""Turns an ncu launch log into the per-launch counters the benchmark reports beside its roofline.

    ncu --metrics dram__bytes_read.sum,dram__bytes_write.sum,smsp__inst_executed.sum,gpu__time_duration.sum \
        --clock-control none -k regex:gemv_stream -s <warm-up launches> -c <launches of one step> \
        --csv --log-file counters.csv python bench.py --profile --steps 2 --warmup 3
    python -m paper_2502_15779_b200.ncu_counters counters.csv llama2_70b_M1_auto

writes (or replaces) the line of that key in profiles/counters.txt: the number of launches captured, the DRAM
bytes (read + written) and the warp instructions per launch, averaged, and a hash of the CUDA sources the
capture was taken from. bench.py reports the figures only while that hash still matches the sources.
"""
import csv
import hashlib
import os
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def source_sha():
    h = hashlib.sha1()
    d = os.path.join(ROOT, "paper_2502_15779_b200", "csrc")
    for name in sorted(os.listdir(d)):
        h.update(name.encode())
        h.update(open(os.path.join(d, name), "rb").read())
    return h.hexdigest()[:16]


def parse(path):
    rows = list(csv.DictReader(ln for ln in open(path) if not ln.startswith("==")))
    per = {}
    for r in rows:
        v = float(r["Metric Value"].replace(",", ""))
        unit = r.get("Metric Unit", "")
        if r["Metric Name"].startswith("dram__bytes") and unit.lower().startswith("k"):
            v *= 1e3
        if r["Metric Name"].startswith("dram__bytes") and unit.lower().startswith("m"):
            v *= 1e6
        per.setdefault(int(r["ID"]), {})[r["Metric Name"]] = v
    n = len(per)
    dram = sum(d.get("dram__bytes_read.sum", 0.0) + d.get("dram__bytes_write.sum", 0.0) for d in per.values()) / n
    inst = sum(d.get("smsp__inst_executed.sum", 0.0) for d in per.values()) / n
    return n, dram, inst


def main():
    path, key = sys.argv[1], sys.argv[2]
    n, dram, inst = parse(path)
    out = os.path.join(ROOT, "profiles", "counters.txt")
    lines = [ln for ln in (open(out).read().splitlines() if os.path.exists(out) else []) if ln.split()[:1] != [key]]
    lines.append(f"{key} launches {n} dram_bytes_per_launch {dram:.0f} warp_instructions_per_launch {inst:.0f} "
                 f"source_sha {source_sha()}")
    open(out, "w").write("\n".join(lines) + "\n")
    print(lines[-1])


if __name__ == "__main__":
    main()
