"""Small helpers that turn ncu's CSV exports into the figures kept under profiles/.

    python -m paper_2407_17353_b200.ncu_summaries traffic <raw.csv> <kernel regex>   # writes profiles/matmul_8192_dram_traffic.json
    python -m paper_2407_17353_b200.ncu_summaries launches <launches.csv>            # prints the per-kernel table

`raw.csv` is `ncu -i <report>.ncu-rep --page raw --csv`; `launches.csv` is the log of
`ncu --metrics gpu__time_duration.sum --csv --log-file ...`.  The traffic record carries a hash of the matmul
kernel's source files, so that bench.py reports the figure only while the kernel is the one that was captured.
"""
import csv
import hashlib
import json
import os
import re
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
MATMUL_SOURCES = ["paper_2407_17353_b200/csrc/matmul_tcgen05.cu", "paper_2407_17353_b200/csrc/tcgen05_ptx.cuh"]


def _num(s):
    return float(s.replace(",", ""))


def traffic(raw_csv, kernel_regex):
    rows = list(csv.reader(open(raw_csv)))
    head, units = rows[0], rows[1]
    col = {k: i for i, k in enumerate(head)}
    scale = {"byte": 1.0, "Kbyte": 1e3, "Mbyte": 1e6, "Gbyte": 1e9}
    out = []
    for r in rows[2:]:
        if not re.search(kernel_regex, r[col["Kernel Name"]]):
            continue
        tot = 0.0
        for m in ("dram__bytes_read.sum", "dram__bytes_write.sum"):
            tot += _num(r[col[m]]) * scale[units[col[m]]]
        out.append(tot)
    if not out:
        raise SystemExit("no launch matches " + kernel_regex)
    h = hashlib.sha256()
    for f in MATMUL_SOURCES:
        h.update(open(os.path.join(ROOT, f), "rb").read())
    rec = {"kernel": kernel_regex, "launches": len(out), "dram_bytes_per_launch": int(sum(out) / len(out)),
           "sources": MATMUL_SOURCES, "sources_sha256": h.hexdigest()}
    path = os.path.join(ROOT, "profiles", "matmul_8192_dram_traffic.json")
    json.dump(rec, open(path, "w"), indent=1)
    print(path, rec)


def launches(log_csv):
    rows = [r for r in csv.reader(open(log_csv)) if len(r) > 10 and r[0].isdigit()]
    agg = {}
    for r in rows:
        name = re.sub(r"\(.*", "", r[4]).replace("void ", "").replace("scalify::", "")
        unit, val = r[-2], _num(r[-1])
        us = val / 1000.0 if unit in ("ns", "nsecond") else (val if unit in ("us", "usecond") else val * 1000.0)
        a = agg.setdefault(name, [0, 0.0])
        a[0] += 1
        a[1] += us
    total = sum(v[1] for v in agg.values())
    print("| kernel | launches | total us | mean us | share |\n|---|---|---|---|---|")
    for name, (n, us) in sorted(agg.items(), key=lambda kv: -kv[1][1]):
        print(f"| `{name}` | {n} | {us:.0f} | {us / n:.1f} | {100 * us / total:.1f} % |")
    print(f"\nSum: {total:.0f} us")


if __name__ == "__main__":
    if len(sys.argv) >= 4 and sys.argv[1] == "traffic":
        traffic(sys.argv[2], sys.argv[3])
    elif len(sys.argv) >= 3 and sys.argv[1] == "launches":
        launches(sys.argv[2])
    else:
        raise SystemExit(__doc__)
