"""Sinks for the library's per-launch and per-event records (observability; no arithmetic of the method).

``write_launch_records`` turns the records of ``Halos.timing_launches()`` (kind, trace events carried out,
algorithmic bytes per parameter, CUDA-event duration) into JSON lines or CSV, one row per kernel launch;
``write_event_log`` does the same for the event log of ``Halos.replay`` (counters, staleness, GPS lag, whether
the event pushed and whether it ran inside a fused launch).
"""
from __future__ import annotations

import csv
import json
from pathlib import Path

import numpy as np

from .binding import KERNEL_NAMES
from .inputs.trace import KIND_NAMES


def _write(path, rows, fields):
    path = Path(path)
    with open(path, "w", newline="") as f:
        if path.suffix == ".csv":
            w = csv.DictWriter(f, fieldnames=fields)
            w.writeheader()
            w.writerows(rows)
        else:
            for r in rows:
                f.write(json.dumps(r) + "\n")
    return len(rows)


def write_launch_records(path, records: np.ndarray, P: int) -> int:
    """One row per timed launch: index, kernel, events, bytes (= bytes_per_param x P), microseconds, GB/s."""
    rows = []
    for n, r in enumerate(records):
        ms = float(r["ms"])
        byts = int(r["bytes_per_param"]) * int(P)
        rows.append({"launch": n, "kernel": KERNEL_NAMES[int(r["kind"])], "events": int(r["events"]),
                     "bytes": byts, "us": ms * 1e3, "GBps": (byts / 1e9 / (ms * 1e-3) if ms > 0 else None)})
    return _write(path, rows, ["launch", "kernel", "events", "bytes", "us", "GBps"])


def write_event_log(path, log: np.ndarray) -> int:
    """One row per replayed event of a ``Halos.replay`` log."""
    fields = ["index", "kind", "lps", "worker", "t", "t_last", "gps_iter", "worker_staleness", "gps_lag", "pushed", "fused"]
    rows = []
    for r in log:
        row = {f: int(r[f]) for f in fields}
        row["kind"] = KIND_NAMES[row["kind"]]
        rows.append(row)
    return _write(path, rows, fields)
