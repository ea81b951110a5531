"""Writes tests/golden/event_log_hashes.txt: for each configured workload the SHA-256 of the event log
(kind, lps, worker, t, t_last, GPS iteration, worker staleness, GPS lag, pushed) that replaying its
seeded trace must produce.  The log is derived from the CPU oracle's counters only; run from the
repository root:   python tests/golden/make_event_log_hashes.py
"""
import sys
from pathlib import Path

HERE = Path(__file__).resolve().parent
sys.path.insert(0, str(HERE.parent))
sys.path.insert(0, str(HERE.parent.parent))

from paper_2506_04531_b200.inputs import workloads  # noqa: E402  (seeded trace generator: inputs only)
from sliced_oracle import log_hash, oracle_event_log  # noqa: E402

NAMES = ("toy", "toy_k4", "70m", "160m", "160m_dn", "410m")

if __name__ == "__main__":
    lines = ["# workload  events  sha256 of the oracle-derived event log (see make_event_log_hashes.py)"]
    for name in NAMES:
        wl = workloads.workload(name)
        ev = wl.trace()
        lines.append(f"{name} {len(ev)} {log_hash(oracle_event_log(wl, ev))}")
    (HERE / "event_log_hashes.txt").write_text("\n".join(lines) + "\n")
    print("\n".join(lines))
