"""The CPU oracle replayed on contiguous index slices in parallel threads.

Every step of the method is elementwise, so replaying a trace on an index range gives exactly that
range of the full result (an invariant pinned in test_oracle_pins.py).  One independent oracle per
slice, each fed by the C twin of the input generator applied to ITS OWN worker snapshots; the C calls
release the GIL, so the slices run on as many cores as the host offers.  Nothing here touches CUDA.
"""
from __future__ import annotations

import concurrent.futures as cf
import hashlib
import os
from typing import Dict, List, Sequence, Tuple

import numpy as np

from oracle import HalosOracle
from paper_2506_04531_b200.inputs import trace as tr
from paper_2506_04531_b200.inputs.gen_c import HostGenerator

LOG_FIELDS = ("kind", "lps", "worker", "t", "t_last", "gps_iter", "worker_staleness", "gps_lag", "pushed")


def host_threads(limit: int = 32) -> int:
    n = len(os.sched_getaffinity(0)) if hasattr(os, "sched_getaffinity") else (os.cpu_count() or 1)
    return max(1, min(limit, n))


def state_buffers(wl) -> List[Tuple[str, int]]:
    """(oracle buffer name, index) of every state buffer of a workload's context."""
    out = [("Theta", 0), ("Mg", 0)]
    for l in range(wl.n_lps):
        out += [(b, l) for b in ("th", "ml", "anchor", "outbox", "inbox")]
    out += [("th0", w) for w in range(wl.n_workers)]
    if wl.optimizer:
        out += [("acc_g", 0)] + [("acc", l) for l in range(wl.n_lps)]
    return out


class SlicedOracle:
    """Oracle state for the index range [lo, hi) of a workload, cut into one slice per thread."""

    def __init__(self, wl, lo: int, hi: int, n_threads: int):
        self.wl, self.lo, self.hi = wl, lo, hi
        n = max(1, min(n_threads, hi - lo))
        self.cuts = [lo + (hi - lo) * k // n for k in range(n + 1)]
        self.hg = HostGenerator(wl.layout, wl.seed)
        self.pool = cf.ThreadPoolExecutor(max_workers=n)
        self.oracles = list(self.pool.map(self._make, range(n)))

    def _make(self, k):
        a, b = self.cuts[k], self.cuts[k + 1]
        return HalosOracle(self.hg.theta_init(a, b), self.wl.worker_lps, worker_dtype=self.wl.worker_dtype, **self.wl.hyper())

    def _advance_one(self, k, events):
        o, a = self.oracles[k], self.cuts[k]
        for ev in events:
            kind, l, w = int(ev["kind"]), int(ev["lps"]), int(ev["worker"])
            if kind == tr.ARRIVE:
                o.arrive(w, self.hg.worker_result(o.buffer("th0", w), w, o.worker_info(w)["round"], a, self.wl.worker_dtype))
            elif kind == tr.GPS_RECV:
                o.gps_recv(l)
            else:
                o.pull(l)

    def advance(self, events) -> None:
        list(self.pool.map(lambda k: self._advance_one(k, events), range(len(self.oracles))))

    def mismatches(self, name: str, idx: int, got: np.ndarray) -> int:
        """Number of slices in which `got` (the values of [lo, hi), fp32 or 16-bit patterns) differs in any bit."""
        def one(k):
            a, b = self.cuts[k] - self.lo, self.cuts[k + 1] - self.lo
            want = self.oracles[k].buffer(name, idx)
            return 0 if np.array_equal(got[a:b].view(np.uint8), want.view(np.uint8)) else 1
        return sum(self.pool.map(one, range(len(self.oracles))))

    def close(self):
        for o in self.oracles:
            o.close()
        self.pool.shutdown()


def oracle_event_log(wl, events) -> Dict[str, np.ndarray]:
    """The log the event-queue driver must produce, derived from the oracle's counters alone (a 4-parameter
    oracle: the bookkeeping does not depend on the values)."""
    o = HalosOracle(np.zeros(4, np.float32), wl.worker_lps, worker_dtype=wl.worker_dtype, **wl.hyper())
    zero = np.zeros(4, np.float32 if wl.worker_dtype == 0 else np.uint16)
    inbox_iter = [0] * wl.n_lps
    n = len(events)
    log = {f: np.zeros(n, np.uint64) for f in LOG_FIELDS}
    for k, ev in enumerate(events):
        kind, l, w = int(ev["kind"]), int(ev["lps"]), int(ev["worker"])
        log["kind"][k], log["lps"][k], log["worker"][k] = kind, l, w
        if kind == tr.ARRIVE:
            log["worker_staleness"][k] = o.counters(l)["t"] - o.worker_info(w)["sched_t"]
            log["pushed"][k] = int(o.arrive(w, zero))
        elif kind == tr.GPS_RECV:
            o.gps_recv(l)
            inbox_iter[l] = o.counters(l)["i"]
        else:
            log["gps_lag"][k] = o.counters(l)["i"] - inbox_iter[l]
            o.pull(l)
        c = o.counters(l)
        log["t"][k], log["t_last"][k], log["gps_iter"][k] = c["t"], c["t_last"], c["i"]
    o.close()
    return log


def log_hash(log, fields: Sequence[str] = LOG_FIELDS) -> str:
    """SHA-256 over the log's fields as little-endian uint64 columns (works for the driver's structured log too)."""
    h = hashlib.sha256()
    for f in fields:
        h.update(np.ascontiguousarray(np.asarray(log[f]).astype("<u8")).tobytes())
    return h.hexdigest()
