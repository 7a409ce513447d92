"""Keeps the hardware counters that ``bench.py`` quotes beside its live timings.

``bench.py`` measures durations itself, but two figures of its roofline objects come from an ncu
capture: the DRAM traffic of a launch (``dram__bytes_read.sum + dram__bytes_write.sum``) and the
executed instructions per element.  This module writes them to ``profiles/ncu_counters.txt`` from a
capture file and reads them back:

    python -m paper_2502_05003_b200.ncu_counters record <report.ncu-rep or raw .csv> \\
        --name quantizer_config2 --kernel 'regex of the kernel name' [--launch 0] \\
        [--elements 12582912] --sources paper_2502_05003_b200/csrc/quest_quantize.cu ... \\
        --command 'the ncu command line that made the capture'

Every record stores a hash of the listed source files and the commit that was checked out.  ``read``
drops a record whose sources have changed since, so a stale counter is never printed as current.
"""
from __future__ import annotations

import argparse
import configparser
import csv
import hashlib
import io
import os
import re
import subprocess

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
DEFAULT_FILE = os.path.join(ROOT, "profiles", "ncu_counters.txt")


def sources_hash(paths) -> str:
    h = hashlib.sha1()
    for p in sorted(paths):
        with open(os.path.join(ROOT, p), "rb") as f:
            h.update(p.encode() + b"\0" + f.read() + b"\0")
    return h.hexdigest()


def _raw_rows(capture: str):
    """Rows of ``ncu --page raw --csv`` for a report file, or of a csv log written by ``ncu --csv``."""
    if capture.endswith(".ncu-rep"):
        text = subprocess.run(["ncu", "-i", capture, "--page", "raw", "--csv"], capture_output=True, text=True,
                              check=True).stdout
    else:
        with open(capture) as f:
            text = f.read()
    lines = [ln for ln in text.splitlines() if ln.startswith('"')]
    return list(csv.reader(io.StringIO("\n".join(lines))))


def _launches(capture: str, kernel_regex: str):
    """Per launch of a matching kernel: {metric name: (value, unit)}.  Handles both csv shapes ncu
    writes: one row per launch with a column per metric (raw page), or one row per metric."""
    rows = _raw_rows(capture)
    if not rows:
        raise SystemExit(f"{capture}: no csv rows")
    hdr = rows[0]
    pat = re.compile(kernel_regex)
    out = []
    if "Metric Name" in hdr:                                  # one row per (launch, metric)
        ki, ii = hdr.index("Kernel Name"), hdr.index("ID")
        mi, ui, vi = hdr.index("Metric Name"), hdr.index("Metric Unit"), hdr.index("Metric Value")
        by_id = {}
        for r in rows[1:]:
            if len(r) <= vi or not pat.search(r[ki]):
                continue
            by_id.setdefault(r[ii], {"_kernel": r[ki]})[r[mi]] = (r[vi], r[ui])
        out = [by_id[k] for k in sorted(by_id, key=lambda s: int(s))]
    else:                                                     # raw page: header, units, then launches
        units = rows[1]
        ki = hdr.index("Kernel Name")
        for r in rows[2:]:
            if len(r) == len(hdr) and pat.search(r[ki]):
                d = {h: (r[i], units[i]) for i, h in enumerate(hdr)}
                d["_kernel"] = r[ki]
                out.append(d)
    return out


def _number(entry) -> float:
    value, unit = entry
    v = float(value.replace(",", ""))
    scale = {"Kbyte": 1e3, "Mbyte": 1e6, "Gbyte": 1e9, "byte": 1.0, "usecond": 1e-6, "us": 1e-6, "msecond": 1e-3,
             "ms": 1e-3, "nsecond": 1e-9, "ns": 1e-9, "second": 1.0}.get(unit, 1.0)
    return v * scale


def record(capture: str, name: str, kernel_regex: str, launch: int, elements: int, sources, command: str,
           path: str = DEFAULT_FILE) -> dict:
    launches = _launches(capture, kernel_regex)
    if not launches:
        raise SystemExit(f"no launch of a kernel matching {kernel_regex!r} in {capture}")
    m = launches[launch]
    rec = {"kernel": m["_kernel"] if isinstance(m["_kernel"], str) else m["_kernel"][0]}
    rec["kernel"] = rec["kernel"][:200]
    if "dram__bytes_read.sum" in m and "dram__bytes_write.sum" in m:
        rec["dram_bytes"] = str(int(round(_number(m["dram__bytes_read.sum"]) + _number(m["dram__bytes_write.sum"]))))
        rec["dram_bytes_read"] = str(int(round(_number(m["dram__bytes_read.sum"]))))
    if "gpu__time_duration.sum" in m:
        rec["duration_us"] = "%.2f" % (_number(m["gpu__time_duration.sum"]) * 1e6)
    if elements and "smsp__thread_inst_executed.sum" in m:
        rec["thread_instructions_per_element"] = "%.2f" % (_number(m["smsp__thread_inst_executed.sum"]) / elements)
    elif elements and "smsp__inst_executed.sum" in m:
        rec["thread_instructions_per_element"] = "%.2f" % (32.0 * _number(m["smsp__inst_executed.sum"]) / elements)
    if elements:
        rec["elements"] = str(elements)
    for key, metric in (("tensor_pipe_active_pct", "sm__pipe_tensor_cycles_active.avg.pct_of_peak_sustained_active"),
                        ("dram_throughput_pct", "gpu__dram_throughput.avg.pct_of_peak_sustained_elapsed"),
                        ("issue_active_pct", "smsp__issue_active.avg.pct")):
        if metric in m:
            rec[key] = "%.1f" % _number(m[metric])
    rec["sources"] = " ".join(sorted(sources))
    rec["sources_sha1"] = sources_hash(sources)
    try:
        rec["captured_at_commit"] = subprocess.run(["git", "-C", ROOT, "rev-parse", "--short", "HEAD"],
                                                   capture_output=True, text=True).stdout.strip() or "unknown"
    except OSError:
        rec["captured_at_commit"] = "unknown"
    rec["command"] = command
    cp = configparser.ConfigParser(interpolation=None)
    if os.path.exists(path):
        cp.read(path)
    cp[name] = rec
    with open(path, "w") as f:
        f.write("# Written by `python -m paper_2502_05003_b200.ncu_counters record`; read by bench.py.\n"
                "# A record is quoted only while the sha1 of its source files still matches.\n")
        cp.write(f)
    return rec


def read(path: str = DEFAULT_FILE, only_current: bool = True) -> dict:
    cp = configparser.ConfigParser(interpolation=None)
    cp.read(path)
    out = {}
    for name in cp.sections():
        sec = dict(cp[name])
        srcs = sec.get("sources", "").split()
        try:
            current = bool(srcs) and sources_hash(srcs) == sec.get("sources_sha1")
        except OSError:
            current = False
        if only_current and not current:
            continue
        rec = {"current": current,
               "source": f"profiles/ncu_counters.txt [{name}] captured at commit {sec.get('captured_at_commit', '?')}"}
        for k in ("dram_bytes", "dram_bytes_read", "elements"):
            if k in sec:
                rec[k] = int(sec[k])
        for k in ("duration_us", "thread_instructions_per_element", "tensor_pipe_active_pct", "dram_throughput_pct",
                  "issue_active_pct"):
            if k in sec:
                rec[k] = float(sec[k])
        out[name] = rec
    return out


def main():
    ap = argparse.ArgumentParser(description=__doc__, formatter_class=argparse.RawDescriptionHelpFormatter)
    sub = ap.add_subparsers(dest="cmd", required=True)
    r = sub.add_parser("record")
    r.add_argument("capture")
    r.add_argument("--name", required=True)
    r.add_argument("--kernel", required=True)
    r.add_argument("--launch", type=int, default=0)
    r.add_argument("--elements", type=int, default=0)
    r.add_argument("--sources", nargs="+", required=True)
    r.add_argument("--command", default="")
    r.add_argument("--file", default=DEFAULT_FILE)
    s = sub.add_parser("show")
    s.add_argument("--file", default=DEFAULT_FILE)
    a = ap.parse_args()
    if a.cmd == "record":
        print(record(a.capture, a.name, a.kernel, a.launch, a.elements, a.sources, a.command, a.file))
    else:
        for k, v in read(a.file, only_current=False).items():
            print(k, v)


if __name__ == "__main__":
    main()
