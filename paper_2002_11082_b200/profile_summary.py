"""Summarises Nsight Compute reports of this library's kernels as text.

    python -m paper_2002_11082_b200.profile_summary counters OUT.md ELEMENTS REPORT.ncu-rep [REPORT ...]
        one table of the counters that matter for a streaming kernel (duration, DRAM bytes and
        throughput, issue and pipe utilisation, occupancy, top stall reasons) per captured launch;
        ELEMENTS is the number of gradient elements one launch processes (for bytes per element).
        With --traffic KEY=KERNEL[,KEY=KERNEL...] the DRAM bytes per element of the named kernels
        are also written to profiles/dram_bytes_per_element.json together with the hash of the
        kernel sources, which is what bench.py reads for `roofline.traffic`.

    python -m paper_2002_11082_b200.profile_summary launches OUT.md LAUNCHES.csv
        per kernel: launches, total time and share, from the CSV log of
        `ncu --metrics gpu__time_duration.sum --csv --log-file LAUNCHES.csv ...`.

Reads reports with `ncu -i REPORT --page raw --csv` (no GPU needed).
"""
from __future__ import annotations

import csv
import hashlib
import io
import json
import os
import re
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

COUNTERS = [
    ("duration us", "gpu__time_duration.sum", 1.0),
    ("DRAM read + write MB", "derived:dram_mb", 1.0),
    ("DRAM throughput % of peak", "gpu__dram_throughput.avg.pct_of_peak_sustained_elapsed", 1.0),
    ("warp instructions", "derived:warp_inst", 1.0),
    ("issue slots busy %", "smsp__issue_active.avg.pct_of_peak_sustained_active", 1.0),
    ("ALU pipe % (active)", "sm__inst_executed_pipe_alu.avg.pct_of_peak_sustained_active", 1.0),
    ("FMA pipe % (active)", "sm__inst_executed_pipe_fma.avg.pct_of_peak_sustained_active", 1.0),
    ("LSU pipe % (active)", "sm__inst_executed_pipe_lsu.avg.pct_of_peak_sustained_active", 1.0),
    ("warps active % of max", "sm__warps_active.avg.pct_of_peak_sustained_active", 1.0),
    ("registers / thread", "launch__registers_per_thread", 1.0),
    ("stall long scoreboard / issue", "smsp__average_warps_issue_stalled_long_scoreboard_per_issue_active.ratio", 1.0),
    ("stall short scoreboard / issue", "smsp__average_warps_issue_stalled_short_scoreboard_per_issue_active.ratio", 1.0),
    ("stall math pipe / issue", "smsp__average_warps_issue_stalled_math_pipe_throttle_per_issue_active.ratio", 1.0),
    ("stall mio throttle / issue", "smsp__average_warps_issue_stalled_mio_throttle_per_issue_active.ratio", 1.0),
    ("stall barrier / issue", "smsp__average_warps_issue_stalled_barrier_per_issue_active.ratio", 1.0),
    ("stall wait / issue", "smsp__average_warps_issue_stalled_wait_per_issue_active.ratio", 1.0),
]


def kernel_sources_hash() -> str:
    h = hashlib.sha256()
    csrc = os.path.join(ROOT, "paper_2002_11082_b200", "csrc")
    for name in sorted(os.listdir(csrc)) + ["../../include/ogq.h"]:
        with open(os.path.join(csrc, name), "rb") as f:
            h.update(name.encode() + b"\0" + f.read())
    return h.hexdigest()


def _to_number(text: str, unit: str) -> float:
    v = float(text.replace(",", ""))
    scale = {"byte": 1e-6, "Kbyte": 1e-3, "Mbyte": 1.0, "Gbyte": 1e3, "ns": 1e-3, "us": 1.0, "ms": 1e3, "s": 1e6}
    return v * scale.get(unit, 1.0)


def read_report(path: str):
    """[(kernel name, {metric: value})] of one report; bytes in MB and times in us."""
    out = subprocess.run(["ncu", "-i", path, "--page", "raw", "--csv"], check=True, capture_output=True, text=True).stdout
    rows = list(csv.reader(io.StringIO(out)))
    hdr, units = rows[0], rows[1]
    name_col = hdr.index("Kernel Name")
    res = []
    for r in rows[2:]:
        vals = {}
        for h, u, v in zip(hdr, units, r):
            if v == "" or h in ("Kernel Name",):
                continue
            try:
                vals[h] = _to_number(v, u)
            except ValueError:
                pass
        # totals the sections give only as rates: DRAM bytes (read + write) and executed warp instructions
        if "dram__bytes_read.sum" in vals:
            vals["derived:dram_mb"] = vals["dram__bytes_read.sum"] + vals.get("dram__bytes_write.sum", 0.0)
        elif "dram__bytes.sum.per_second" in vals:
            unit = units[hdr.index("dram__bytes.sum.per_second")]
            per_s = float(r[hdr.index("dram__bytes.sum.per_second")].replace(",", "")) * {"Tbyte/s": 1e12, "Gbyte/s": 1e9, "Mbyte/s": 1e6}.get(unit, 1.0)
            vals["derived:dram_mb"] = per_s * vals["gpu__time_duration.sum"] * 1e-6 / 1e6
        if "smsp__inst_executed.sum" in vals:
            vals["derived:warp_inst"] = vals["smsp__inst_executed.sum"]
        elif "sm__inst_executed.sum.per_cycle_elapsed" in vals and "gpc__cycles_elapsed.max" in vals:
            vals["derived:warp_inst"] = vals["sm__inst_executed.sum.per_cycle_elapsed"] * vals["gpc__cycles_elapsed.max"]
        res.append((r[name_col], vals))
    return res


def short(name: str) -> str:
    m = re.search(r"(k_[a-z0-9_]+)(<[^>]*>)?", name)
    return (m.group(1) + (m.group(2) or "")) if m else name[:60]


def cmd_counters(argv):
    traffic_keys = {}
    if "--traffic" in argv:
        i = argv.index("--traffic")
        for kv in argv[i + 1].split(","):
            k, v = kv.split("=")
            traffic_keys[v] = k
        argv = argv[:i] + argv[i + 2:]
    out_md, elements, reports = argv[0], float(argv[1]), argv[2:]
    cols = []
    for rep in reports:
        for name, vals in read_report(rep):
            cols.append((short(name), os.path.basename(rep), vals))
    lines = ["| counter | " + " | ".join(f"{n} ({r})" for n, r, _ in cols) + " |", "|---|" + "---|" * len(cols)]
    for label, metric, _ in COUNTERS:
        cells = []
        for _, _, vals in cols:
            v = vals.get(metric)
            cells.append("" if v is None else (f"{v:,.0f}" if abs(v) >= 1000 else f"{v:.3g}"))
        lines.append(f"| {label} | " + " | ".join(cells) + " |")
    per_elem, instr = [], []
    for _, _, vals in cols:
        mb = vals.get("derived:dram_mb", 0.0)
        per_elem.append(f"{mb * 1e6 / elements:.3f}")
        wi = vals.get("derived:warp_inst")
        instr.append("" if wi is None else f"{wi * 32 / elements:.1f}")
    lines.append("| DRAM bytes / element | " + " | ".join(per_elem) + " |")
    lines.append("| thread instructions / element | " + " | ".join(instr) + " |")
    with open(out_md, "a") as f:
        f.write("\n".join(lines) + "\n")
    if traffic_keys:
        path = os.path.join(ROOT, "profiles", "dram_bytes_per_element.json")
        rec = {"sources_sha256": kernel_sources_hash(), "entries": {}}
        if os.path.exists(path):
            old = json.load(open(path))
            if old.get("sources_sha256") == rec["sources_sha256"]:
                rec["entries"] = old.get("entries", {})
        for name, _, vals in cols:
            base = re.sub(r"<.*", "", name)
            for kern, key in traffic_keys.items():
                if base == re.sub(r"<.*", "", kern) or name == kern:
                    mb = vals.get("derived:dram_mb", 0.0)
                    rec["entries"][key] = round(mb * 1e6 / elements, 4)
        json.dump(rec, open(path, "w"), indent=1, sort_keys=True)


def cmd_launches(argv):
    out_md, log = argv
    text = open(log).read()
    start = text.index('"ID"')
    rows = list(csv.DictReader(io.StringIO(text[start:])))
    agg = {}
    for r in rows:
        if r.get("Metric Name") != "gpu__time_duration.sum":
            continue
        v = _to_number(r["Metric Value"], r["Metric Unit"])
        n = short(r["Kernel Name"])
        t, c = agg.get(n, (0.0, 0))
        agg[n] = (t + v, c + 1)
    total = sum(t for t, _ in agg.values()) or 1.0
    lines = ["| kernel | launches | total us | mean us | share |", "|---|---|---|---|---|"]
    for n, (t, c) in sorted(agg.items(), key=lambda kv: -kv[1][0]):
        lines.append(f"| {n} | {c} | {t:.1f} | {t / c:.1f} | {t / total:.3f} |")
    with open(out_md, "a") as f:
        f.write("\n".join(lines) + "\n")


if __name__ == "__main__":
    if len(sys.argv) < 3 or sys.argv[1] not in ("counters", "launches"):
        raise SystemExit(__doc__)
    (cmd_counters if sys.argv[1] == "counters" else cmd_launches)(sys.argv[2:])
