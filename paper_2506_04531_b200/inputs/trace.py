"""Integer-time generator of asynchronous event traces (harness, not part of the update path).

It is the paper's trace-driven simulator (Appendix A, "Simulation methodology") reduced to
what fixes the ORDER of server-side updates: point-to-point transfers take size/bandwidth
(the alpha-beta model with zero propagation delay), a worker round takes
download + H * T_profiled * S_fastest / S + upload, servers process instantly, and ties are
broken by (time, kind, lps, worker) with ARRIVE < GPS_RECV < PULL.  All times are integer
nanoseconds, so the order is reproducible everywhere.

Event kinds
    ARRIVE(w)     a worker's result reaches its LPS                 (Alg. 1 line 9)
    GPS_RECV(l)   the Delta pushed by LPS l reaches the GPS          (Alg. 1 line 2)
    PULL(l)       the Theta_i sent back reaches LPS l                (Alg. 1 line 17)
A push happens inside the ARRIVE that completes a window of K updates (Alg. 1 line 13); the
generator tracks only the counters it needs to know when that is.
"""
from __future__ import annotations

import heapq
from dataclasses import dataclass, field
from typing import List, Optional, Sequence

import numpy as np

ARRIVE, GPS_RECV, PULL = 0, 1, 2
KIND_NAMES = ("ARRIVE", "GPS_RECV", "PULL")

EVENT_DTYPE = np.dtype([("kind", np.uint8), ("lps", np.uint8), ("worker", np.uint16),
                        ("pad", np.uint32), ("time_ns", np.int64)])

# Inter-region bandwidths to region R-1, where the GPS sits (Gbps; the paper's bandwidth table,
# first row) and the intra-region bandwidth.
GBPS_TO_GPS_REGION = (100.0, 0.537, 0.935, 0.202)
GBPS_INTRA = 100.0
H_LOCAL_STEPS = 8
# Relative speeds of the paper's 16 workers, four per region (its worker-speed table).
PAPER_WORKER_SPEEDS = (10.0, 9.1, 3.8, 2.6, 9.4, 8.0, 6.3, 5.8, 9.9, 5.7, 2.1, 1.5, 9.1, 8.7, 5.8, 1.2)

_M64 = (1 << 64) - 1


def _splitmix64(state: int):
    state = (state + 0x9E3779B97F4A7C15) & _M64
    z = state
    z = ((z ^ (z >> 30)) * 0xBF58476D1CE4E5B9) & _M64
    z = ((z ^ (z >> 27)) * 0x94D049BB133111EB) & _M64
    return state, z ^ (z >> 31)


def worker_speeds(n_workers: int, seed: int, lo: float = 1.0, hi: float = 4.0) -> List[float]:
    """Relative speeds drawn uniformly in [lo, hi] from a seeded integer generator."""
    out, st = [], seed & _M64
    for _ in range(n_workers):
        st, r = _splitmix64(st)
        out.append(lo + (hi - lo) * ((r >> 11) / float(1 << 53)))
    return out


def transfer_ns(n_bytes: int, gbps: float) -> int:
    return int(round(n_bytes * 8.0 / gbps))  # bits / (Gbit/s) = ns


@dataclass
class TraceSpec:
    P: int
    worker_lps: Sequence[int]
    speeds: Sequence[float]
    t_profiled_ms: float
    n_arrivals: int
    K: int = 32
    bytes_per_param: int = 4
    lps_gbps: Optional[Sequence[float]] = None   # LPS -> GPS bandwidth; default by region
    h_steps: int = H_LOCAL_STEPS
    dyn_updates: bool = False        # dynamic local updates: H scaled with worker speed, so that all
                                     # workers finish a round in the time the fastest needs for H steps
    bandwidth_scale: float = 1.0     # multiplies every link bandwidth (the paper's 2x-bandwidth study)


def generate_trace(spec: TraceSpec) -> np.ndarray:
    """Returns the total order of events as a structured array of EVENT_DTYPE."""
    n_workers = len(spec.worker_lps)
    n_lps = max(spec.worker_lps) + 1
    lps_gbps = list(spec.lps_gbps) if spec.lps_gbps is not None else [
        GBPS_TO_GPS_REGION[l % len(GBPS_TO_GPS_REGION)] for l in range(n_lps)]
    model_bytes = spec.P * spec.bytes_per_param
    hop = transfer_ns(model_bytes, GBPS_INTRA * spec.bandwidth_scale)
    s_max = max(spec.speeds)
    if spec.dyn_updates:
        # H_w = H * S_w / S_max local steps, each taking T_prof * S_max / S_w: every round costs H * T_prof
        round_ns = [2 * hop + int(round(spec.h_steps * spec.t_profiled_ms * 1e6)) for _ in spec.speeds]
    else:
        round_ns = [2 * hop + int(round(spec.h_steps * spec.t_profiled_ms * 1e6 * s_max / s))
                    for s in spec.speeds]
    link_ns = [transfer_ns(model_bytes, g * spec.bandwidth_scale) for g in lps_gbps]

    heap = [(round_ns[w], ARRIVE, spec.worker_lps[w], w) for w in range(n_workers)]
    heapq.heapify(heap)
    t = [0] * n_lps
    t_last = [0] * n_lps
    in_flight = [False] * n_lps
    events, arrivals = [], 0
    while heap:
        now, kind, l, w = heapq.heappop(heap)
        if kind == ARRIVE:
            if arrivals >= spec.n_arrivals:
                continue  # the trace stops admitting arrivals; round trips in flight still drain
            arrivals += 1
            events.append((kind, l, w, 0, now))
            t[l] += 1
            heapq.heappush(heap, (now + round_ns[w], ARRIVE, l, w))
            if t[l] - t_last[l] == spec.K:
                assert not in_flight[l]
                in_flight[l] = True
                heapq.heappush(heap, (now + link_ns[l], GPS_RECV, l, 0))
        elif kind == GPS_RECV:
            events.append((kind, l, 0, 0, now))
            heapq.heappush(heap, (now + link_ns[l], PULL, l, 0))
        else:
            events.append((kind, l, 0, 0, now))
            t_last[l] = t[l]
            in_flight[l] = False
    return np.array(events, dtype=EVENT_DTYPE)


def random_trace(n_workers_lps: Sequence[int], n_events: int, K: int, seed: int) -> np.ndarray:
    """A valid but otherwise arbitrary event order for small tests (no timing model):
    at each step one of the currently legal events is picked by a seeded generator."""
    n_lps = max(n_workers_lps) + 1
    t, t_last = [0] * n_lps, [0] * n_lps
    phase = [0] * n_lps
    st = seed & _M64
    events = []
    for n in range(n_events):
        legal = [(ARRIVE, n_workers_lps[w], w) for w in range(len(n_workers_lps))]
        for l in range(n_lps):
            if phase[l] == 1:
                legal += [(GPS_RECV, l, 0)] * 2
            elif phase[l] == 2:
                legal += [(PULL, l, 0)] * 2
        st, r = _splitmix64(st)
        kind, l, w = legal[r % len(legal)]
        events.append((kind, l, w, 0, n))
        if kind == ARRIVE:
            t[l] += 1
            if t[l] - t_last[l] == K:
                phase[l] = 1
        elif kind == GPS_RECV:
            phase[l] = 2
        else:
            phase[l] = 0
            t_last[l] = t[l]
    return np.array(events, dtype=EVENT_DTYPE)


def save_trace(path, events: np.ndarray) -> None:
    """Trace file = the flat little-endian array of 16-byte records {u8 kind, u8 lps, u16 worker, u32 pad,
    i64 time_ns}; the same layout the C driver takes."""
    np.ascontiguousarray(events, dtype=EVENT_DTYPE).tofile(str(path))


def load_trace(path) -> np.ndarray:
    ev = np.fromfile(str(path), dtype=EVENT_DTYPE)
    if ev.size and int(ev["kind"].max()) > PULL:
        raise ValueError("not a trace file: unknown event kind")
    return ev
