"""Turns ncu CSV output into the short text summaries kept under profiles/.

    python -m paper_2501_07161_b200.ncu_summary launches <launch-list.csv>
        per kernel: launches, total and average device time, share of the total; DRAM bytes when
        the capture holds dram__bytes_read.sum / dram__bytes_write.sum
    python -m paper_2501_07161_b200.ncu_summary raw <raw-page.csv> [metric substring ...]
        one block per captured launch with the counters the profiles quote (or those named)
    python -m paper_2501_07161_b200.ncu_summary traffic <launch-list.csv> <kernel substring> <algorithmic bytes> <out.txt> [note]
        DRAM bytes per algorithmic byte of one kernel, written together with a hash of the kernel
        sources so that a reader (bench.py) can tell whether the record still describes the code

The launch-list CSV is what `ncu --csv --log-file F --metrics ...` writes; the raw page is
`ncu -i report.ncu-rep --page raw --csv`.
"""
from __future__ import annotations

import collections
import csv
import hashlib
import os
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
TRAFFIC_SOURCES = ["paper_2501_07161_b200/csrc/qv2_metrics.cu", "paper_2501_07161_b200/csrc/qv2_device.cuh",
                   "paper_2501_07161_b200/csrc/qv2_common.cuh"]
DEFAULT_RAW = ["gpu__time_duration.sum", "dram__bytes_read.sum", "dram__bytes_write.sum",
               "gpu__dram_throughput.avg.pct_of_peak_sustained_elapsed",
               "sm__warps_active.avg.pct_of_peak_sustained_active", "launch__registers_per_thread",
               "launch__grid_size", "smsp__issue_active.avg.pct_of_peak_sustained_active",
               "sm__pipe_alu_cycles_active.avg.pct_of_peak_sustained_active",
               "sm__pipe_fma_cycles_active.avg.pct_of_peak_sustained_active",
               "l1tex__data_bank_conflicts_pipe_lsu_mem_shared_op_atom.sum", "lts__t_sector_hit_rate.pct",
               "sm__cycles_active.avg", "sm__cycles_active.max", "sm__cycles_elapsed.max",
               "sm__pipe_tensor_cycles_active.avg.pct_of_peak_sustained_active"]

_TIME = {"ns": 1e-3, "nsecond": 1e-3, "us": 1.0, "usecond": 1.0, "ms": 1e3, "msecond": 1e3, "s": 1e6, "second": 1e6}
_BYTES = {"byte": 1.0, "Kbyte": 1e3, "Mbyte": 1e6, "Gbyte": 1e9}


def _num(text: str) -> float:
    return float(text.replace(",", "") or 0.0)


def _short(name: str) -> str:
    return name.split("(")[0].replace("void ", "").replace("unnamed>::", "")


def read_launch_list(path: str):
    """-> ordered dict launch id -> {"name": kernel, metric: value}; times in microseconds, bytes in bytes."""
    with open(path) as f:
        lines = [ln for ln in f if not ln.startswith("==")]
    launches = collections.OrderedDict()
    for row in csv.DictReader(lines):
        d = launches.setdefault(row["ID"], {"name": _short(row["Kernel Name"])})
        v, unit = _num(row["Metric Value"]), row["Metric Unit"]
        d[row["Metric Name"]] = v * (_TIME.get(unit, 1.0) if "time" in row["Metric Name"] else _BYTES.get(unit, 1.0))
    return launches


def by_kernel(launches):
    agg = collections.OrderedDict()
    for d in launches.values():
        a = agg.setdefault(d["name"], collections.Counter())
        a["launches"] += 1
        for k, v in d.items():
            if k != "name":
                a[k] += v
    return agg


def cmd_launches(path: str) -> str:
    agg = by_kernel(read_launch_list(path))
    has_time = any("gpu__time_duration.sum" in a for a in agg.values())
    key = "gpu__time_duration.sum" if has_time else "dram__bytes_read.sum"
    total = sum(a[key] for a in agg.values())
    out = []
    for name, a in sorted(agg.items(), key=lambda kv: -kv[1][key]):
        line = "%-40s launches=%4d" % (name[:40], a["launches"])
        if has_time:
            t = a["gpu__time_duration.sum"]
            line += " total_us=%10.1f avg_us=%9.2f share=%5.1f%%" % (t, t / a["launches"], 100.0 * t / total)
        if "dram__bytes_read.sum" in a:
            line += "  dram_read_MB/launch=%9.2f" % (a["dram__bytes_read.sum"] / a["launches"] / 1e6)
        if "dram__bytes_write.sum" in a:
            line += "  dram_write_MB/launch=%7.2f" % (a["dram__bytes_write.sum"] / a["launches"] / 1e6)
        out.append(line)
    if has_time:
        out.append("total device time of the listed launches: %.1f us" % total)
    if any("dram__bytes_read.sum" in a for a in agg.values()):
        out.append("total DRAM bytes read by the listed launches: %.1f MB" %
                   (sum(a.get("dram__bytes_read.sum", 0.0) for a in agg.values()) / 1e6))
    return "\n".join(out)


def cmd_raw(path: str, wanted) -> str:
    rows = list(csv.reader(open(path)))
    hdr, units, data = rows[0], rows[1], rows[2:]
    idx = {h: i for i, h in enumerate(hdr)}
    wanted = wanted or DEFAULT_RAW
    out = []
    for d in data:
        out.append(_short(d[idx["Kernel Name"]]))
        for h in hdr:
            if any(h == w or (w not in DEFAULT_RAW and w in h) for w in wanted):
                out.append("  %-72s %s %s" % (h, d[idx[h]], units[idx[h]]))
        stalls = []
        for h in hdr:
            if h.startswith("smsp__average_warps_issue_stalled_") and h.endswith("_per_issue_active.ratio"):
                v = _num(d[idx[h]])
                if v >= 0.3:
                    stalls.append((v, h[len("smsp__average_warps_issue_stalled_"):-len("_per_issue_active.ratio")]))
        out.append("  warps stalled per issue: " + ", ".join("%s %.2f" % (n, v) for v, n in sorted(stalls, reverse=True)))
    return "\n".join(out)


def sources_hash() -> str:
    h = hashlib.sha256()
    for rel in TRAFFIC_SOURCES:
        with open(os.path.join(ROOT, rel), "rb") as f:
            h.update(f.read())
    return h.hexdigest()


def cmd_traffic(path: str, kernel: str, algorithmic_bytes: float, out_path: str, note: str = "") -> str:
    agg = by_kernel(read_launch_list(path))
    match = [(n, a) for n, a in agg.items() if kernel in n]
    if len(match) != 1:
        raise SystemExit("kernel substring must match exactly one kernel, got %r" % [n for n, _ in match])
    name, a = match[0]
    dram = (a["dram__bytes_read.sum"] + a.get("dram__bytes_write.sum", 0.0)) / a["launches"]
    text = "\n".join([
        "# DRAM traffic of %s per launch, from the ncu capture summarised beside this file;" % name,
        "# bench.py scales it to its own launch by the algorithmic bytes and reports it as roofline.traffic",
        "# only while the sources listed below still hash to sha256.  %s" % note,
        "dram_bytes_per_launch: %d" % dram,
        "algorithmic_bytes_per_launch: %d" % algorithmic_bytes,
        "dram_bytes_per_algorithmic_byte: %.6f" % (dram / algorithmic_bytes),
        "sources: " + " ".join(TRAFFIC_SOURCES),
        "sha256: " + sources_hash(), ""])
    with open(out_path, "w") as f:
        f.write(text)
    return text


def main(argv):
    if len(argv) >= 2 and argv[0] == "launches":
        print(cmd_launches(argv[1]))
    elif len(argv) >= 2 and argv[0] == "raw":
        print(cmd_raw(argv[1], argv[2:]))
    elif len(argv) >= 5 and argv[0] == "traffic":
        print(cmd_traffic(argv[1], argv[2], float(argv[3]), argv[4], " ".join(argv[5:])))
    else:
        raise SystemExit(__doc__)


if __name__ == "__main__":
    main(sys.argv[1:])
