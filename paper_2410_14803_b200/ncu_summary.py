"""Turns Nsight Compute output into the short records kept under ``profiles/``.

    # launch list (per kernel: launches, total time, share) from
    #   ncu --metrics gpu__time_duration.sum --clock-control none --csv --log-file launches.csv <cmd>
    python -m paper_2410_14803_b200.ncu_summary launches launches.csv

    # DRAM traffic of one call (read + written bytes of the kernels that make it up) from
    #   ncu -i prof.ncu-rep --page raw --csv > raw.csv
    # written into profiles/traffic.json, which bench.py reads for `roofline.traffic`
    python -m paper_2410_14803_b200.ncu_summary traffic raw.csv --workload large \\
        --kernels "scan_mask_kernel|scan_pipe_kernel" --command "<the capture command>" [--scale 16]

    # a few named counters per kernel from the same raw.csv
    python -m paper_2410_14803_b200.ncu_summary counters raw.csv

The traffic record carries a hash of the kernel sources it was measured with, so that a number taken
from an older kernel is never reported beside a newer one.
"""
from __future__ import annotations

import argparse
import csv
import hashlib
import json
import os
import re
import sys
from collections import OrderedDict

_PKG = os.path.dirname(os.path.abspath(__file__))
_ROOT = os.path.dirname(_PKG)
TRAFFIC_JSON = os.path.join(_ROOT, "profiles", "traffic.json")

_UNIT = {"byte": 1.0, "Kbyte": 1e3, "Mbyte": 1e6, "Gbyte": 1e9, "Tbyte": 1e12,
         "ns": 1e-3, "us": 1.0, "ms": 1e3, "s": 1e6, "usecond": 1.0, "nsecond": 1e-3, "msecond": 1e3, "second": 1e6}

COUNTERS = ["gpu__time_duration.sum", "dram__bytes_read.sum", "dram__bytes_write.sum",
            "gpu__dram_throughput.avg.pct_of_peak_sustained_elapsed", "launch__registers_per_thread",
            "sm__warps_active.avg.pct_of_peak_sustained_active", "smsp__inst_executed.sum",
            "smsp__average_warps_issue_stalled_long_scoreboard_per_issue_active.ratio",
            "smsp__average_warps_issue_stalled_barrier_per_issue_active.ratio",
            "smsp__average_warps_issue_stalled_short_scoreboard_per_issue_active.ratio",
            "smsp__average_warps_issue_stalled_membar_per_issue_active.ratio",
            "smsp__average_warps_issue_stalled_wait_per_issue_active.ratio",
            "sm__inst_issued.avg.pct_of_peak_sustained_active"]


def kernel_sources_sha256(names=None) -> str:
    """Hash of the named kernel source files under csrc/ (default: all of them), in name order."""
    h = hashlib.sha256()
    d = os.path.join(_PKG, "csrc")
    for name in sorted(names if names else os.listdir(d)):
        if name.endswith((".cu", ".cuh")):
            h.update(name.encode())
            with open(os.path.join(d, name), "rb") as f:
                h.update(f.read())
    return h.hexdigest()


def short_name(kernel: str) -> str:
    k = re.sub(r"^void\s+", "", kernel)
    k = re.sub(r"\(.*$", "", k)
    return k.replace("distrl::", "")


def _csv_rows(path):
    with open(path, newline="") as f:
        lines = [ln for ln in f if ln.startswith('"')]
    return list(csv.reader(lines))


def read_launches(path):
    """[(kernel, microseconds)] from a `--metrics gpu__time_duration.sum --csv` log."""
    rows = _csv_rows(path)
    head = rows[0]
    ik, im, iu, iv = (head.index(c) for c in ("Kernel Name", "Metric Name", "Metric Unit", "Metric Value"))
    out = []
    for r in rows[1:]:
        if r[im] == "gpu__time_duration.sum":
            out.append((short_name(r[ik]), float(r[iv].replace(",", "")) * _UNIT.get(r[iu], 1.0)))
    return out


def read_raw(path):
    """[(kernel, {metric: value in base units (bytes, microseconds, or as printed)})] from `--page raw --csv`."""
    rows = _csv_rows(path)
    head, units = rows[0], rows[1]
    ik = head.index("Kernel Name")
    out = []
    for r in rows[2:]:
        vals = {}
        for name, unit, v in zip(head, units, r):
            try:
                vals[name] = float(v.replace(",", "")) * _UNIT.get(unit, 1.0)
            except ValueError:
                pass
        out.append((short_name(r[ik]), vals))
    return out


def launches_table(path) -> str:
    agg = OrderedDict()
    for k, us in read_launches(path):
        c = agg.setdefault(k, [0, 0.0])
        c[0] += 1
        c[1] += us
    total = sum(v[1] for v in agg.values()) or 1.0
    lines = ["| kernel | launches | total us | avg us | share |", "|---|---|---|---|---|"]
    for k, (cnt, us) in sorted(agg.items(), key=lambda kv: -kv[1][1]):
        lines.append("| %s | %d | %.1f | %.2f | %.1f %% |" % (k, cnt, us, us / cnt, 100.0 * us / total))
    return "\n".join(lines)


def counters_table(path) -> str:
    per = OrderedDict()
    for k, vals in read_raw(path):
        per.setdefault(k, []).append(vals)
    names = [c for c in COUNTERS if any(c in v for vs in per.values() for v in vs)]
    lines = ["| counter | " + " | ".join(per) + " |", "|---" * (len(per) + 1) + "|"]
    for c in names:
        cells = []
        for vs in per.values():
            xs = [v[c] for v in vs if c in v]
            cells.append("%.4g" % (sum(xs) / len(xs)) if xs else "")
        lines.append("| %s | %s |" % (c, " | ".join(cells)))
    lines.append("(bytes in bytes, times in microseconds, averaged over %s captured launches per kernel)"
                 % "/".join(str(len(v)) for v in per.values()))
    return "\n".join(lines)


def traffic_record(path, kernels: str, scale: float, sources):
    pat = re.compile(kernels)
    per = OrderedDict()
    for k, vals in read_raw(path):
        if pat.search(k) and "dram__bytes_read.sum" in vals:
            per.setdefault(k, []).append(vals["dram__bytes_read.sum"] + vals["dram__bytes_write.sum"])
    if not per:
        raise SystemExit("no kernel matches %r" % kernels)
    kern = {k: scale * sum(v) / len(v) for k, v in per.items()}
    return {"bytes_per_call": int(round(sum(kern.values()))),
            "kernels": {k: int(round(v)) for k, v in kern.items()},
            "launches_captured": {k: len(v) for k, v in per.items()},
            "scaled_by": scale, "sources": sorted(sources), "source_sha256": kernel_sources_sha256(sources)}


def main(argv=None):
    ap = argparse.ArgumentParser(description=__doc__, formatter_class=argparse.RawDescriptionHelpFormatter)
    sub = ap.add_subparsers(dest="what", required=True)
    a = sub.add_parser("launches")
    a.add_argument("csv")
    a = sub.add_parser("counters")
    a.add_argument("csv")
    a = sub.add_parser("traffic")
    a.add_argument("csv")
    a.add_argument("--workload", required=True)
    a.add_argument("--kernels", required=True, help="regular expression over the short kernel names of one call")
    a.add_argument("--scale", type=float, default=1.0, help="units of a full launch / units of the captured one")
    a.add_argument("--sources", default="retrace.cu,common.cuh,priority.cuh,sampler.cuh",
                   help="files under csrc/ that the captured kernels are compiled from")
    a.add_argument("--command", default="", help="the capture command, kept in the record")
    a.add_argument("--note", default="")
    args = ap.parse_args(argv)
    if args.what == "launches":
        print(launches_table(args.csv))
    elif args.what == "counters":
        print(counters_table(args.csv))
    else:
        rec = traffic_record(args.csv, args.kernels, args.scale, [x for x in args.sources.split(",") if x])
        rec["command"] = args.command
        if args.note:
            rec["note"] = args.note
        try:
            with open(TRAFFIC_JSON) as f:
                allrec = json.load(f)
        except Exception:
            allrec = {}
        allrec[args.workload] = rec
        with open(TRAFFIC_JSON, "w") as f:
            json.dump(allrec, f, indent=1, sort_keys=True)
            f.write("\n")
        print(json.dumps(rec, indent=1))
    return 0


if __name__ == "__main__":
    sys.exit(main())
