"""Hardware counters of the library's kernels, recorded for ONE revision of their sources.

Some figures cannot be measured by a timing run: the warp instructions a kernel executes and the bytes it
moves to and from DRAM come from a profiler capture.  They are stored in `counters.json` beside this file
together with a hash of the sources the kernel is built from; `lookup()` returns them with `stale: True`
once any of those sources has changed, so that a report never shows counters of a kernel that no longer
exists.

Recording (after a profiler run that wrote a CSV with the metrics smsp__inst_executed.sum,
l1tex__data_pipe_lsu_wavefronts_mem_shared.sum, dram__bytes_read.sum and dram__bytes_write.sum of one launch):

    python -m paper_2408_00741_b200.counters record --kernel eval_select_kernel --workload cfg4 \
        --csv capture.csv --units 64 --evals 1698693120 --command "<the profiler command>"

`units` is what the launch processed in the unit the traffic grows with (scenarios for the sweep,
requests for the binning); `evals` the candidates (or requests) it evaluated.
"""
from __future__ import annotations

import argparse
import csv
import hashlib
import json
import os

_HERE = os.path.dirname(os.path.abspath(__file__))
PATH = os.path.join(_HERE, "counters.json")

# the sources each kernel is compiled from (relative to this package)
SOURCES = {
    "eval_select_kernel": ("csrc/sweep.cu", "csrc/eval_dev.cuh", "csrc/dyn_internal.cuh"),
    "bin_trace_kernel": ("csrc/bin_trace.cu", "csrc/dyn_internal.cuh"),
    "bin_tokens_kernel": ("csrc/tokens.cu", "csrc/dyn_internal.cuh"),
}


def source_hash(kernel: str) -> str:
    h = hashlib.sha256()
    for rel in SOURCES[kernel]:
        with open(os.path.join(_HERE, rel), "rb") as fh:
            h.update(fh.read())
    return h.hexdigest()[:16]


def _load() -> dict:
    try:
        with open(PATH) as fh:
            return json.load(fh)
    except (OSError, ValueError):
        return {}


def lookup(kernel: str, workload: str):
    """The recorded counters of `kernel` on `workload`, or None.  `stale` tells whether the kernel's
    sources have changed since they were taken."""
    rec = _load().get(f"{kernel}/{workload}")
    if rec is None:
        return None
    out = dict(rec)
    out["stale"] = rec.get("sources_sha256_16") != source_hash(kernel)
    return out


def parse_csv(path: str) -> dict:
    """Metric name -> value summed over the rows of a profiler CSV (one captured launch)."""
    vals: dict = {}
    with open(path, newline="") as fh:
        rows = [r for r in csv.reader(fh) if r]
    header = next(r for r in rows if "Metric Name" in r)
    i_name, i_unit, i_val = header.index("Metric Name"), header.index("Metric Unit"), header.index("Metric Value")
    scale = {"byte": 1.0, "Kbyte": 1e3, "Mbyte": 1e6, "Gbyte": 1e9, "inst": 1.0, "": 1.0}
    for r in rows[rows.index(header) + 1:]:
        if len(r) <= i_val:
            continue
        try:
            v = float(r[i_val].replace(",", ""))
        except ValueError:
            continue
        vals[r[i_name]] = vals.get(r[i_name], 0.0) + v * scale.get(r[i_unit], 1.0)
    return vals


def record(kernel: str, workload: str, csv_path: str, units: float, evals: float, command: str) -> dict:
    m = parse_csv(csv_path)
    rec = {
        "sources_sha256_16": source_hash(kernel),
        "units": units, "evals": evals,
        "warp_instructions": m.get("smsp__inst_executed.sum"),
        "shared_wavefronts": m.get("l1tex__data_pipe_lsu_wavefronts_mem_shared.sum"),
        "dram_bytes_read": m.get("dram__bytes_read.sum"),
        "dram_bytes_written": m.get("dram__bytes_write.sum"),
        "command": command,
    }
    if rec["warp_instructions"] is not None:
        rec["warp_inst_per_32_evals"] = rec["warp_instructions"] * 32.0 / evals
    if rec["shared_wavefronts"] is not None:
        rec["shared_wavefronts_per_32_evals"] = rec["shared_wavefronts"] * 32.0 / evals
    if rec["dram_bytes_read"] is not None and rec["dram_bytes_written"] is not None:
        rec["dram_bytes_per_unit"] = (rec["dram_bytes_read"] + rec["dram_bytes_written"]) / units
    allrec = _load()
    allrec[f"{kernel}/{workload}"] = rec
    with open(PATH, "w") as fh:
        json.dump(allrec, fh, indent=1, sort_keys=True)
        fh.write("\n")
    return rec


if __name__ == "__main__":
    ap = argparse.ArgumentParser()
    ap.add_argument("action", choices=["record", "show"])
    ap.add_argument("--kernel")
    ap.add_argument("--workload")
    ap.add_argument("--csv")
    ap.add_argument("--units", type=float)
    ap.add_argument("--evals", type=float)
    ap.add_argument("--command", default="")
    a = ap.parse_args()
    if a.action == "record":
        print(json.dumps(record(a.kernel, a.workload, a.csv, a.units, a.evals, a.command), indent=1))
    else:
        for k in sorted(_load()):
            kern, wl = k.split("/")
            print(k, json.dumps(lookup(kern, wl)))
