"""DRAM traffic per launch of the softmax workloads, from ncu's launch lists.

The record lives in ``profiles/dram_traffic.txt`` (text, one line per workload); ``bench.py`` reads it
for ``roofline.traffic``. It is written by this module from the CSV logs of

    ncu --metrics dram__bytes_read.sum,dram__bytes_write.sum --print-units base --clock-control none \
        --cache-control none -k regex:<kernel> -s <warm-up launches> -c 8 --csv --log-file <log>.csv \
        python bench.py --workload cfgN [--rows R] --steps 8 --trains 1 --warmup 3 --no-all --no-e2e --no-cpu --no-clocks

(one capture per workload, after the same command has exited 0 without ncu): eight CONSECUTIVE launches
over the rotating buffer pairs, so that the lines a launch leaves dirty in the write-back L2 are counted
when the following launches evict them; a single isolated launch ends before most of y has reached DRAM
and under-counts the write half. The eight launches are summed and divided by eight. Where the capture
used only the first R rows of a workload (cfg5: 2048 of 32768, a full 8 GiB launch is not captured), the
figure is scaled by rows / R: traffic is proportional to the rows processed.

    python -m paper_2607_24762_b200.traffic --out profiles/dram_traffic.txt cfg2=log_cfg2.csv cfg5=log_cfg5.csv:2048 ...
"""
from __future__ import annotations

import argparse
import csv
import datetime

from . import workloads as W


def parse_log(path: str):
    """Sum of dram__bytes_read.sum and dram__bytes_write.sum over the launches of an ncu --csv log.
    Returns (kernel name, launches, read bytes, write bytes)."""
    rows = []
    with open(path, newline="") as f:
        lines = [ln for ln in f if ln.startswith('"')]
    for rec in csv.DictReader(lines):
        rows.append(rec)
    rd = wr = 0.0
    ids = set()
    kernel = ""
    for r in rows:
        name, val = r.get("Metric Name", ""), r.get("Metric Value", "").replace(",", "")
        if name not in ("dram__bytes_read.sum", "dram__bytes_write.sum") or not val:
            continue
        unit = r.get("Metric Unit", "byte")
        if unit != "byte":
            raise ValueError(f"{path}: expected base units (--print-units base), got {unit!r}")
        ids.add(r["ID"])
        kernel = r["Kernel Name"].split("(")[0].split("<")[0].replace("void ", "")
        if name.startswith("dram__bytes_read"):
            rd += float(val)
        else:
            wr += float(val)
    if not ids:
        raise ValueError(f"{path}: no dram__bytes_* rows")
    return kernel, len(ids), int(rd), int(wr)


def write(out_path: str, specs: list[str]) -> None:
    lines = ["# DRAM bytes per launch of fs_softmax on the five workloads: ncu dram__bytes_read.sum + dram__bytes_write.sum,",
             "# summed over 8 consecutive launches on rotating buffers and divided by 8 (see paper_2607_24762_b200/traffic.py",
             "# for the capture command). Columns: workload kernel launches rows_captured rows read_bytes write_bytes",
             "# bytes_per_launch (scaled to the full workload) algorithmic_bytes ratio",
             f"# written {datetime.date.today().isoformat()}"]
    for spec in specs:
        name, rest = spec.split("=", 1)
        path, _, cap = rest.partition(":")
        w = W.WORKLOADS[name]
        cap_rows = int(cap) if cap else w.rows
        kernel, n, rd, wr = parse_log(path)
        per = (rd + wr) / n * (w.rows / cap_rows)
        lines.append(f"{name} {kernel} {n} {cap_rows} {w.rows} {rd} {wr} {int(per)} {w.min_bytes} {per / w.min_bytes:.4f}")
    with open(out_path, "w") as f:
        f.write("\n".join(lines) + "\n")


def read(path: str) -> dict:
    """{workload: {"bytes_per_launch": int, "note": str}} from the record written by `write`."""
    out = {}
    with open(path) as f:
        for ln in f:
            if ln.startswith("#") or not ln.strip():
                continue
            name, kernel, n, cap_rows, rows, rd, wr, per, alg, ratio = ln.split()
            note = (f"ncu dram__bytes_read.sum + dram__bytes_write.sum of {kernel}, mean of {n} consecutive launches"
                    + (f" of the first {cap_rows} rows, scaled to {rows}" if cap_rows != rows else "")
                    + " (profiles/dram_traffic.txt)")
            out[name] = {"bytes_per_launch": int(per), "note": note}
    return out


if __name__ == "__main__":
    ap = argparse.ArgumentParser()
    ap.add_argument("--out", required=True)
    ap.add_argument("specs", nargs="+", help="cfgN=ncu_log.csv[:rows_captured]")
    a = ap.parse_args()
    write(a.out, a.specs)
    print(open(a.out).read())
