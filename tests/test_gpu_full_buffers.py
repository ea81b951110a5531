"""EVERY element of EVERY state buffer of the LLM-shaped configurations, CUDA against the oracle.

The CUDA side replays the configured seeded trace at full size through the batched event-queue driver
(halos_replay_batched, up to 8 arrivals and GPS+merge pairs fused per launch).  The oracle replays the
same trace on contiguous index slices, one per host core (tests/sliced_oracle.py).  At several
checkpoints and at the end every buffer is copied back and compared bit for bit; the driver's event
log is compared with the log derived from the oracle's counters, and its hash with the stored one.

Host memory: the oracle's state for an index range is ~(2 + 7 LPS + workers) arrays of that range; when
that does not fit comfortably the index range is covered in several passes, each with its own CUDA
replay from the initial state (the replay is seconds; the oracle dominates).
"""
from __future__ import annotations

import time
from pathlib import Path

import numpy as np
import psutil
import pytest
import torch

from paper_2506_04531_b200 import binding as hb
from paper_2506_04531_b200.inputs import gen, trace as tr, workloads
from paper_2506_04531_b200.inputs.gen_cuda import DeviceGenerator
from sliced_oracle import LOG_FIELDS, SlicedOracle, host_threads, log_hash, oracle_event_log, state_buffers

pytestmark = pytest.mark.gpu

_BUF = {"Theta": hb.BUF_THETA_G, "Mg": hb.BUF_M_G, "th": hb.BUF_THETA_L, "ml": hb.BUF_M_L, "anchor": hb.BUF_ANCHOR,
        "outbox": hb.BUF_OUTBOX, "inbox": hb.BUF_INBOX, "th0": hb.BUF_THETA0, "acc": hb.BUF_ACC_L, "acc_g": hb.BUF_ACC_G}
GOLDEN = Path(__file__).parent / "golden" / "event_log_hashes.txt"
ORACLE_TIME_LIMIT_S = 400      # per test; the default-suite tests need 25 s (70m), 140 s (160m) and 190 s (410m) on 16 cores


@pytest.fixture(scope="module", autouse=True)
def _built():
    from paper_2506_04531_b200 import build
    build.build()


def _golden_hash(name):
    for line in GOLDEN.read_text().splitlines():
        if line and not line.startswith("#") and line.split()[0] == name:
            return int(line.split()[1]), line.split()[2]
    raise KeyError(name)


def _every_element(name: str, n_events, n_checkpoints: int, need_device_gb: float):
    wl = workloads.workload(name)
    lay, P = wl.layout, wl.layout.P
    torch.cuda.empty_cache()
    free, _ = torch.cuda.mem_get_info()
    if free < need_device_gb * (1 << 30):
        pytest.skip(f"needs ~{need_device_gb:.0f} GB of free device memory")
    events_all = wl.trace()
    events = events_all if n_events is None else events_all[:n_events]
    # Keep the oracle's time bounded on hosts with few cores: it replays ~150 M parameter-events per second and core
    # (measured; generator included).  On the 16-core hosts of this machine nothing is cut.
    threads = host_threads(32)
    affordable = int(ORACLE_TIME_LIMIT_S * threads * 150e6 / P)
    if len(events) > affordable:
        print(f"[{name}] {threads} host cores: trace cut from {len(events)} to {affordable} events to stay within {ORACLE_TIME_LIMIT_S} s of oracle time")
        events, n_events = events[:affordable], affordable
    n = len(events)
    checkpoints = sorted({n * (k + 1) // (n_checkpoints + 1) for k in range(n_checkpoints)} | {n})
    names = state_buffers(wl)
    wbytes = 4 if wl.worker_dtype == gen.F32 else 2
    tdt = torch.float32 if wl.worker_dtype == gen.F32 else torch.int16

    # host memory plan: oracle state per parameter (fp32 master arrays incl. the oracle's two extra per LPS, worker copies)
    per_param = 4 * (3 + 7 * wl.n_lps) + wbytes * wl.n_workers + 8
    budget = 0.45 * psutil.virtual_memory().available
    passes = max(1, int(np.ceil(per_param * P / budget)))
    ranges = [(P * k // passes, P * (k + 1) // passes) for k in range(passes)]

    dg = DeviceGenerator(lay, wl.seed)
    bufs = [torch.empty(P, dtype=tdt, device="cuda") for _ in range(wl.n_workers)]   # a result lives until its worker's next
    pinned = torch.empty(max(hi - lo for lo, hi in ranges) * 4, dtype=torch.uint8, pin_memory=True)
    want_log = oracle_event_log(wl, events)
    t_gpu = t_cpu = 0.0
    compared = 0
    for lo, hi in ranges:
        h = hb.Halos(dg.theta_init(), wl.worker_lps, lay.numel, worker_dtype=wl.worker_dtype, **wl.hyper())

        def producer(index, worker, rnd):
            return dg.worker_result(h.peek(hb.BUF_THETA0, worker), worker, rnd, out=bufs[worker], worker_dtype=wl.worker_dtype)

        so = SlicedOracle(wl, lo, hi, threads)
        logs, prev = [], 0
        for cp in checkpoints:
            t0 = time.perf_counter()
            logs.append(h.replay(events[prev:cp], producer, max_batch=8))
            torch.cuda.synchronize()
            t_gpu += time.perf_counter() - t0
            t0 = time.perf_counter()
            so.advance(events[prev:cp])
            t_cpu += time.perf_counter() - t0
            bad = []
            for bname, idx in names:
                dev = h.peek(_BUF[bname], idx)[lo:hi]
                nbytes = dev.numel() * dev.element_size()
                host = pinned[:nbytes]
                host.copy_(dev.contiguous().view(torch.uint8))
                torch.cuda.synchronize()
                bits16 = bname == "th0" and wl.worker_dtype == gen.BF16
                if so.mismatches(bname, idx, host.numpy().view(np.uint16 if bits16 else np.float32)):
                    bad.append((bname, idx, cp))
                compared += dev.numel()
            assert not bad, bad[:8]
            prev = cp
        # the driver's own log of this replay against the oracle-derived one
        log = np.concatenate(logs)
        for f in LOG_FIELDS:
            assert np.array_equal(log[f].astype(np.uint64), want_log[f]), f
        assert log_hash(log) == log_hash(want_log)
        assert h.batch_info()["multi_launches"] > 0 and int(log["fused"].sum()) > 0
        so.close()
        h.close()
        del h
        torch.cuda.empty_cache()
    if n_events is None:                      # the whole configured trace: its stored hash
        assert (n, log_hash(want_log)) == _golden_hash(name)
    assert compared == len(names) * P * len(checkpoints)
    print(f"[{name}] {n} events, {len(names)} buffers x {P} elements x {len(checkpoints)} checkpoints bit-identical; "
          f"{passes} pass(es), {threads} oracle threads, CUDA replay {t_gpu:.1f} s, oracle {t_cpu:.1f} s")


def test_config_70m_bf16_every_element_full_trace():
    """Configuration 2: all 1,052 events, all 20 buffers, 4 checkpoints + the end."""
    _every_element("70m", None, 4, need_device_gb=8)


def test_config_160m_fp32_every_element_full_trace():
    """Configuration 3 (the fp32 headline configuration): all 2,094 events, all 38 buffers, 4 checkpoints + the end."""
    _every_element("160m", None, 4, need_device_gb=40)


def test_config_410m_fp32_every_element():
    """Configuration 4 (the largest): the first 1,100 events -- at least two push/merge round trips at every LPS,
    the slow region's included -- all 54 buffers, 2 checkpoints + the end."""
    wl = workloads.workload("410m")
    ev = wl.trace()[:1100]
    for l in range(wl.n_lps):
        assert int(((ev["kind"] == tr.PULL) & (ev["lps"] == l)).sum()) >= 2
    _every_element("410m", 1100, 2, need_device_gb=150)


def test_config_410m_event_log_hash_from_the_driver():
    """Configuration 4, the whole trace: the staleness order is replayed identically -- the log returned by
    halos_replay_batched (kind, lps, worker, t, t_last, i, worker staleness, GPS lag, pushed) equals the log
    derived from the oracle's counters, field by field and by its stored SHA-256."""
    wl = workloads.workload("410m")
    lay, P = wl.layout, wl.layout.P
    torch.cuda.empty_cache()
    free, _ = torch.cuda.mem_get_info()
    if free < 150 * (1 << 30):
        pytest.skip("needs ~145 GB of free device memory")
    events = wl.trace()
    dg = DeviceGenerator(lay, wl.seed)
    h = hb.Halos(dg.theta_init(), wl.worker_lps, lay.numel, worker_dtype=wl.worker_dtype, **wl.hyper())
    bufs = [torch.empty(P, dtype=torch.float32, device="cuda") for _ in range(wl.n_workers)]
    log = h.replay(events, lambda i, w, r: dg.worker_result(h.peek(hb.BUF_THETA0, w), w, r, out=bufs[w]), max_batch=8)
    torch.cuda.synchronize()
    want = oracle_event_log(wl, events)
    for f in LOG_FIELDS:
        assert np.array_equal(log[f].astype(np.uint64), want[f]), f
    assert (len(events), log_hash(log)) == _golden_hash("410m")
    assert bool(torch.isfinite(h.peek(hb.BUF_THETA_G)).all())
    # with several workers per LPS every LPS sees stale results
    arr = log["kind"] == tr.ARRIVE
    mean_stale = [float(log["worker_staleness"][arr & (log["lps"] == l)].mean()) for l in range(wl.n_lps)]
    assert all(m > 0 for m in mean_stale)
    h.close()


# ---------------------------------------------------------------------------------------------
# Longer runs of the same check, outside the default suite's time budget: HALOS_LONG_TESTS=1 enables them.
# ---------------------------------------------------------------------------------------------
_LONG = pytest.mark.skipif(__import__("os").environ.get("HALOS_LONG_TESTS") != "1",
                           reason="set HALOS_LONG_TESTS=1 (adds ~8 minutes of oracle time on 16 cores)")


@_LONG
def test_config_410m_fp32_every_element_whole_trace():
    """Configuration 4 over its WHOLE trace (2,094 events), all 54 buffers, 2 checkpoints + the end."""
    _every_element("410m", None, 2, need_device_gb=150)


@_LONG
def test_config_160m_delayed_nesterov_every_element():
    """The 160M configuration under the delayed-Nesterov optimizer with the paper's selected values (d_l = 16,
    d_g = 2): the first 800 events (fused launches with refreshes inside batches, GPS refreshes, merges), all 43
    buffers including the accumulators, 2 checkpoints + the end."""
    _every_element("160m_dn", 800, 2, need_device_gb=45)
