#!/usr/bin/env python
"""Benchmark of the HALoS server-side update path on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload 160m] [--impl ours|reference]

A step replays the next ``--events-per-step`` events (worker arrivals with their pushes, GPS
updates, merges) of the workload's seeded asynchronous trace through the library's event-queue
driver.  Metric: parameters updated per second (every event updates the P parameters of one model).
Worker results are the faithful theta_H = theta_0 + noise of every arrival: the timed steps are run
once untimed with the generator in the loop, each result is kept in HBM, the state is rebuilt and
the timed runs read the resident results (and must end in the same state, which is checked).  The
step length is reduced from 128 events until the results of all timed steps fit in device memory.

    value       device-resident: every arrival's result theta_H already sits in HBM; the driver fuses up to
                --max-batch arrivals at one LPS into one launch (bit-identical to one launch per
                event, which is measured too and reported under per_event_kernels)
    e2e         the same replay through the C ABI with HOST-resident worker results (pinned), the
                host->device copy of every result and a device->host read of a probe of the
                models inside the timed region
    roofline    arrive kernel (delta + LPS momentum + schedule copy): algorithmic bytes / mean
                launch duration (CUDA events recorded by the library on its stream inside the timed
                region) against the measured HBM copy bandwidth of this machine
    cpu_baseline  the CPU oracle as it stands (one core) on a bounded index slice of the workload

``--impl reference`` times the CPU oracle on a bounded sample and prints the same line shape.
With N > 1 (torchrun) every rank replays the trace on its own index shard of an N-times larger
model on its own GPU: no data-path collective; NCCL only carries the barrier and the max of the
per-rank times.
"""
from __future__ import annotations

import argparse
import json
import os
import sys
import threading
import time
from pathlib import Path

import numpy as np

ROOT = Path(__file__).resolve().parent
if str(ROOT) not in sys.path:
    sys.path.insert(0, str(ROOT))

METRIC = "params_updated_per_sec"
UNIT = "params/s"
BYTES_PER_PARAM = {"arrive_f32": 28, "arrive_bf16": 22, "arrive_push_f32": 36, "arrive_push_bf16": 30,
                   "push": 12, "gps": 24, "pull": 16, "gps_pull": 36}

# DRAM bytes ncu attributes to a launch = its algorithmic bytes minus the dirty lines still in L2 when the kernel
# ends: 55-60 MB per launch whatever the kernel and the size (one-pass captures of every launch of the 160M bench
# workload and of the 70M-size case; reads equal the algorithmic bytes exactly).
L2_WRITE_RESIDUE_BYTES = 58e6


# ------------------------------------------------------------------------------------ helpers
def measured_peak_gbs():
    p = ROOT / "MEASURED_PEAKS.json"
    if p.exists():
        try:
            return float(json.loads(p.read_text())["hbm_gbs"]), "measured"
        except Exception:
            pass
    return 6650.0, "fallback"


class ClockSampler:
    """Samples SM clock and throttle reasons with NVML while the timed region runs (read-only)."""

    def __init__(self, index: int, period_s: float = 0.2):
        self.index, self.period = index, period_s
        self.samples, self.reasons = [], set()
        self.max_mhz = None
        self._stop = threading.Event()
        self._thr = None
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.dev = None
            try:
                import torch
                uuid = str(torch.cuda.get_device_properties(index).uuid)
                if not uuid.startswith("GPU-"):
                    uuid = "GPU-" + uuid
                self.dev = pynvml.nvmlDeviceGetHandleByUUID(uuid.encode())
            except Exception:
                self.dev = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = int(pynvml.nvmlDeviceGetMaxClockInfo(self.dev, pynvml.NVML_CLOCK_SM))
        except Exception:
            self.nv = None

    def _names(self, mask: int):
        nv = self.nv
        table = [("gpu_idle", "nvmlClocksThrottleReasonGpuIdle"),
                 ("applications_clocks_setting", "nvmlClocksThrottleReasonApplicationsClocksSetting"),
                 ("sw_power_cap", "nvmlClocksThrottleReasonSwPowerCap"),
                 ("hw_slowdown", "nvmlClocksThrottleReasonHwSlowdown"),
                 ("sync_boost", "nvmlClocksThrottleReasonSyncBoost"),
                 ("sw_thermal_slowdown", "nvmlClocksThrottleReasonSwThermalSlowdown"),
                 ("hw_thermal_slowdown", "nvmlClocksThrottleReasonHwThermalSlowdown"),
                 ("hw_power_brake_slowdown", "nvmlClocksThrottleReasonHwPowerBrakeSlowdown"),
                 ("display_clock_setting", "nvmlClocksThrottleReasonDisplayClockSetting")]
        return {n for n, attr in table if mask & int(getattr(nv, attr, 0))}

    def _run(self):
        while not self._stop.is_set():
            try:
                self.samples.append(int(self.nv.nvmlDeviceGetClockInfo(self.dev, self.nv.NVML_CLOCK_SM)))
                self.reasons |= self._names(int(self.nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.dev)))
            except Exception:
                pass
            self._stop.wait(self.period)

    def __enter__(self):
        if self.nv is not None:
            self._thr = threading.Thread(target=self._run, daemon=True)
            self._thr.start()
        return self

    def __exit__(self, *exc):
        self._stop.set()
        if self._thr:
            self._thr.join()

    def summary(self):
        if not self.samples:
            return {"sm_mhz": None, "sm_max_mhz": self.max_mhz, "reasons": ["unavailable"]}
        return {"sm_mhz": float(np.median(self.samples)), "sm_max_mhz": self.max_mhz,
                "reasons": sorted(self.reasons - {"gpu_idle"})}


def reduce_over_ranks(dist, elapsed_ms: float, units: float, device=None):
    """(max elapsed over ranks, sum of units over ranks); identity without a process group."""
    if dist is None or not dist.is_initialized() or dist.get_world_size() == 1:
        return elapsed_ms, units
    import torch
    t = torch.tensor([elapsed_ms], dtype=torch.float64, device=device)
    u = torch.tensor([units], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    dist.all_reduce(u, op=dist.ReduceOp.SUM)
    return float(t.item()), float(u.item())


def window_events(n_steps: int, events_per_step: int, wl):
    """A trace long enough for n_steps windows of events_per_step events."""
    need = n_steps * events_per_step
    n_arr = max(wl.n_arrivals, need)
    ev = wl.trace(n_arr)
    while len(ev) < need:
        n_arr = int(n_arr * 1.2) + 16
        ev = wl.trace(n_arr)
    return ev[:need]


# ------------------------------------------------------------------------------------ CPU oracle leg
class OracleReplayer:
    """The CPU oracle (as it stands, one core) replaying events on the index slice [0, slice_params) of a
    workload; state persists across calls so that consecutive trace windows can be fed one by one.
    Only the oracle calls are timed (the synthetic inputs are generated outside the timed spans)."""

    def __init__(self, wl, slice_params: int):
        from oracle import HalosOracle
        from paper_2506_04531_b200.inputs import gen
        self.wl, self.lay = wl, wl.layout
        from paper_2506_04531_b200.inputs.gen_c import HostGenerator
        self.S = min(slice_params, self.lay.P)
        self.hg = HostGenerator(self.lay, wl.seed)
        init = self.hg.theta_init(0, self.S)
        self.o = HalosOracle(init, wl.worker_lps, worker_dtype=wl.worker_dtype, dtype=np.float32, **wl.hyper())
        self.by_kind = {}

    def run(self, events, budget_s: float = float("inf")):
        """Returns (seconds spent inside the oracle, events done); self.by_kind accumulates [events, seconds] per kind."""
        from paper_2506_04531_b200.inputs import gen, trace as tr
        o, wl = self.o, self.wl
        spent, done = 0.0, 0
        for ev in events:
            kind, l, w = int(ev["kind"]), int(ev["lps"]), int(ev["worker"])
            if kind == tr.ARRIVE:
                r = o.worker_info(w)["round"]
                thH = self.hg.worker_result(o.buffer("th0", w), w, r, 0, wl.worker_dtype)   # untimed input
                t0 = time.perf_counter()
                pushed = o.arrive(w, thH)
                name = "arrive_push" if pushed else "arrive"
            elif kind == tr.GPS_RECV:
                t0 = time.perf_counter()
                o.gps_recv(l)
                name = "gps"
            else:
                t0 = time.perf_counter()
                o.pull(l)
                name = "pull"
            dt = time.perf_counter() - t0
            spent += dt
            done += 1
            acc = self.by_kind.setdefault(name, [0, 0.0])
            acc[0] += 1
            acc[1] += dt
            if spent >= budget_s:
                break
        return spent, done

    def kind_rates(self):
        """params/s per event kind from everything run so far."""
        return {k: {"events": n, "value": n * self.S / t, "unit": UNIT} for k, (n, t) in sorted(self.by_kind.items()) if t > 0}

    def close(self):
        self.o.close()


def oracle_sample_all_cores(wl, events, slice_params: int, budget_s: float):
    """The same oracle on every core the process may use: one independent replayer per core, each on its
    own copy of the slice (the method is elementwise, so a split by index range needs no communication).
    Returns (aggregate params/s, cores)."""
    import concurrent.futures as cf
    cores = len(os.sched_getaffinity(0)) if hasattr(os, "sched_getaffinity") else (os.cpu_count() or 1)
    reps = [OracleReplayer(wl, slice_params) for _ in range(cores)]
    with cf.ThreadPoolExecutor(max_workers=cores) as ex:
        out = list(ex.map(lambda r: r.run(events, budget_s), reps))   # ctypes releases the GIL inside the oracle
    rate = sum(done * r.S / spent for r, (spent, done) in zip(reps, out) if spent > 0)
    for r in reps:
        r.close()
    return rate, cores


def oracle_sample(wl, events, slice_params: int, budget_s: float, want_kinds: bool = False):
    """Times the oracle from a fresh state on the first events of a trace until the time budget is used.
    Returns (params/s, description, seconds, events[, rates per event kind])."""
    rep = OracleReplayer(wl, slice_params)
    spent, done = rep.run(events, budget_s)
    S = rep.S
    kinds = rep.kind_rates()
    rep.close()
    out = (done * S / spent, f"first {done} events of the trace on the index slice [0,{S}) of {wl.layout.P} parameters", spent, done)
    return out + (kinds,) if want_kinds else out


def run_cpu_table(args):
    """Oracle rates per event kind for every configuration: one core, and one replayer per core, each on bounded
    index slices of the configured trace (CPU only; the core count is printed with the numbers)."""
    from paper_2506_04531_b200.inputs import workloads
    rows = {}
    for name in ("toy", "70m", "160m", "410m"):
        wl = workloads.workload(name)
        ev = wl.trace()
        budget = args.cpu_budget_s
        rate, desc, spent, done, kinds = oracle_sample(wl, ev, 1 << 21, budget, want_kinds=True)
        # long enough to contain pushes, GPS updates and merges: if the budget ended before the first round trip,
        # time those kinds on the events around it
        if "gps" not in kinds or "pull" not in kinds:
            rep = OracleReplayer(wl, 1 << 18)
            rep.run(ev[:min(len(ev), 400)])
            small = rep.kind_rates()
            rep.close()
            for k in ("arrive_push", "gps", "pull"):
                if k not in kinds and k in small:
                    kinds[k] = dict(small[k], note="from a 256K-parameter slice")
        all_rate, cores = oracle_sample_all_cores(wl, ev, 1 << 20, min(8.0, budget))
        rows[name] = {"P": wl.layout.P, "one_core": {"value": rate, "unit": UNIT, "sample": desc + f" ({spent:.1f} s)"},
                      "per_event_kind_one_core": kinds, "all_cores": {"value": all_rate, "cores": cores}}
    print(json.dumps({"cpu_table": rows, "metric": METRIC, "kind": "oracle"}))
    return 0


# ------------------------------------------------------------------------------------ bandwidth sweep
def run_sweep(args):
    """Configuration 5: flat fp32 buffers from 2^20 to 2^30 parameters plus the 1.4B-class decoder layout;
    per size one context with 1 LPS / 1 worker, cycles of {arrive, arrive+due, push, gps, pull, arrive, arrive+due, push,
    gps+pull}, each kernel
    timed by the library's CUDA events.  Sizes whose working set is below 512 MB rotate over several
    contexts so that consecutive launches do not find their data in L2."""
    import torch
    from paper_2506_04531_b200 import binding as hb, build as _build
    from paper_2506_04531_b200.inputs import gen, layouts, workloads
    _build.build()
    dev = torch.device("cuda", 0)
    peak, peak_kind = measured_peak_gbs()
    cases = [(f"flat_{n}", layouts.flat_layout("flat", n)) for n in workloads.SWEEP_SIZES]
    cases.append(("decoder_1p4b", layouts.named_layout("1p4b")))
    rows = []
    for wdt, wname in ((gen.F32, "f32"), (gen.BF16, "bf16")):
        for name, lay in cases:
            P = lay.P
            if args.sweep_max and P > args.sweep_max:
                continue
            wb = 4 if wdt == gen.F32 else 2
            set_bytes = P * (6 * 4 + 3 * wb)
            n_sets = max(1, min(64, -(-(512 << 20) // set_bytes)))
            ctxs, ths = [], []
            for k in range(n_sets):
                init = torch.randn(P, device=dev) * 0.02
                ctxs.append(hb.Halos(init, [0], lay.numel, K=2, worker_dtype=wdt, chunk_elems=args.chunk_elems))
                th = init + 1e-3 * torch.randn(P, device=dev)
                ths.append(th if wdt == gen.F32 else th.to(torch.bfloat16).view(torch.int16))
                del init, th

            def a1(h, th):
                h.worker_delta(0, th); h.lps_apply(0, 0)

            def a2(h, th):
                h.worker_delta(0, th)
                assert h.lps_apply(0, 0)

            phases = (a1, a2, lambda h, th: h.lps_push(0), lambda h, th: h.gps_merge(0), lambda h, th: h.lps_pull(0),
                      a1, a2, lambda h, th: h.lps_push(0), lambda h, th: h.gps_merge_pull(0))

            def cycle():
                # kind-major order: between two launches on the same context all other contexts run,
                # so small sizes do not find their buffers in L2
                for ph in phases:
                    for h, th in zip(ctxs, ths):
                        ph(h, th)

            reps = max(3, min(40, int(2e9 // max(1, P * n_sets))))
            cycle()
            torch.cuda.synchronize(dev)
            for h in ctxs:
                h.timing_enable(True)
            for _ in range(reps):
                cycle()
            agg = {}
            for h in ctxs:
                for k, (n, ms) in h.timing_read().items():
                    a = agg.setdefault(k, [0, 0.0]); a[0] += n; a[1] += ms
                h.close()
            B = {"arrive": 16 + 3 * wb, "push": 12, "gps": 24, "pull": 16, "gps_pull": 36}
            row = {"case": name, "P": P, "tensors": lay.n_tensors, "worker_dtype": wname, "buffer_MB": P * 4 / 1e6,
                   "contexts_rotated": n_sets}
            for k in ("arrive", "push", "gps", "pull", "gps_pull"):
                n, ms = agg[k]
                t = ms / n * 1e-3
                row[k] = {"us": t * 1e6, "GBps": B[k] * P / 1e9 / t, "frac_of_measured": B[k] * P / 1e9 / t / peak,
                          "Gparams_per_s": P / t / 1e9}
            rows.append(row)
            del ctxs, ths
            torch.cuda.empty_cache()
    print(json.dumps({"sweep": rows, "peak_GBps": peak, "peak_source": peak_kind, "metric": METRIC}))
    return 0


# ------------------------------------------------------------------------------------ end-to-end leg
def pcie_ceiling(torch, dev, nbytes: int, reps: int = 6):
    """Pinned host<->device copies of one result's size, both directions at once on two streams (the shape of the
    end-to-end leg): GB/s per direction.  Plain cudaMemcpyAsync through torch, no library code."""
    hin = torch.empty(nbytes, dtype=torch.uint8, pin_memory=True)
    hout = torch.empty(nbytes, dtype=torch.uint8, pin_memory=True)
    din = torch.empty(nbytes, dtype=torch.uint8, device=dev)
    dout = torch.empty(nbytes, dtype=torch.uint8, device=dev)
    s1, s2 = torch.cuda.Stream(dev), torch.cuda.Stream(dev)
    out = {}
    for label, both in (("one_direction", False), ("both_directions", True)):
        for timed in (False, True):
            torch.cuda.synchronize(dev)
            t0 = time.perf_counter()
            for _ in range(reps if timed else 1):
                with torch.cuda.stream(s1):
                    din.copy_(hin, non_blocking=True)
                if both:
                    with torch.cuda.stream(s2):
                        hout.copy_(dout, non_blocking=True)
            torch.cuda.synchronize(dev)
            dt = time.perf_counter() - t0
        out["h2d_GBps_" + label] = reps * nbytes / 1e9 / dt
    torch.cuda.synchronize(dev)
    t0 = time.perf_counter()
    for _ in range(reps):
        with torch.cuda.stream(s2):
            hout.copy_(dout, non_blocking=True)
    torch.cuda.synchronize(dev)
    out["d2h_GBps_one_direction"] = reps * nbytes / 1e9 / (time.perf_counter() - t0)
    return out


def run_e2e(args, wl, hb, tr, torch, dist, dev, fresh_context, timed_events, arrive_slots, resident, eps, K, P, wbytes, wdt):
    """The timed steps through the C ABI with HOST buffers: every arrival's result is copied in from pinned host
    memory (halos_worker_delta_host) and every arrival's answer -- the model its worker restarts from -- is copied
    out to pinned host memory (halos_worker_fetch_host); both copies are inside the timed region.  Covers as many
    of the K steps as fit the pinned-memory budget (min(128 GB, 60% of the free host memory))."""
    import psutil
    ranks_here = int(os.environ.get("LOCAL_WORLD_SIZE", os.environ.get("WORLD_SIZE", "1")))   # ranks sharing this host's memory
    budget = int(min(128 << 30, 0.6 * psutil.virtual_memory().available / max(1, ranks_here)))
    per_step = max(1, sum(1 for i in arrive_slots if i < eps))
    steps = int(max(1, min(K, budget // (wbytes * P) // per_step)))
    n_arr = sum(1 for i in arrive_slots if i < steps * eps)
    host_results = torch.empty((n_arr, P), dtype=wdt, pin_memory=True)   # allocated pinned: no pageable twin
    host_results.copy_(resident[:n_arr])
    ring = [torch.empty(P, dtype=wdt, pin_memory=True) for _ in range(4)]   # answers: a worker consumes its own at once
    ceiling = pcie_ceiling(torch, dev, wbytes * P)
    h = fresh_context()
    torch.cuda.synchronize(dev)
    if dist is not None:
        dist.barrier()
    t0 = time.perf_counter()
    n_out = 0
    for s in range(steps):
        win = timed_events[s * eps:(s + 1) * eps]
        # results are copied in by the library; two staging buffers let the copy of the next result
        # overlap the current update kernel, so up to two results are registered ahead
        order = [k for k in range(len(win)) if int(win[k]["kind"]) == tr.ARRIVE]
        ahead, fed = [], 0

        def feed():
            nonlocal fed
            while fed < len(order) and len(ahead) < 2:
                k = order[fed]
                w = int(win[k]["worker"])
                if any(int(win[p]["worker"]) == w for p in ahead):
                    break
                h.worker_delta_host(w, host_results[arrive_slots[s * eps + k]])
                ahead.append(k)
                fed += 1
        for k in range(len(win)):
            feed()
            kind, l, w = int(win[k]["kind"]), int(win[k]["lps"]), int(win[k]["worker"])
            if kind == tr.ARRIVE:
                assert ahead and ahead[0] == k
                ahead.pop(0)
                if h.lps_apply(l, w):
                    h.lps_push(l)
                h.worker_fetch_host(w, ring[n_out % len(ring)])      # the step's result for this worker
                n_out += 1
            elif kind == tr.GPS_RECV:
                h.gps_merge(l)
            else:
                h.lps_pull(l)
    h.fetch_sync()
    torch.cuda.synchronize(dev)
    dt_ms = (time.perf_counter() - t0) * 1e3
    u = float(steps * eps) * P
    dt_ms, u_all = reduce_over_ranks(dist, dt_ms, u, dev)
    h2d = int(n_arr / steps * P * wbytes)
    d2h = int(n_out / steps * P * wbytes)
    e2e = {"value": u_all / (dt_ms * 1e-3), "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
           "steps": steps, "ms_per_step": dt_ms / steps,
           "what": "worker results from pinned host memory in, each worker's new start model to pinned host memory out"}
    e2e["h2d_GBps"] = h2d / (e2e["ms_per_step"] * 1e6)
    e2e["d2h_GBps"] = d2h / (e2e["ms_per_step"] * 1e6)
    e2e["pcie_ceiling"] = ceiling      # plain pinned copies of one result's size, measured beside it
    e2e["frac_of_pcie_ceiling"] = e2e["h2d_GBps"] / ceiling["h2d_GBps_both_directions"]
    h.close()
    del host_results, ring
    return e2e


# ------------------------------------------------------------------------------------ other configurations
def config_kernel_table(name, args, torch, dev, peak):
    """Per-kernel CUDA-event figures for a whole configured trace (every event, generator in the loop between
    launches, L2 flushed after each generated input), once with one launch per event and once through the fused
    driver.  The library's per-launch events do not need resident inputs."""
    from paper_2506_04531_b200 import binding as hb
    from paper_2506_04531_b200.inputs import gen, workloads
    from paper_2506_04531_b200.inputs.gen_cuda import DeviceGenerator
    wl = workloads.workload(name)
    lay, P = wl.layout, wl.layout.P
    wbytes = 4 if wl.worker_dtype == gen.F32 else 2
    wdt = torch.float32 if wl.worker_dtype == gen.F32 else torch.int16
    need = (2 + 5 * wl.n_lps) * 4 * P + 2 * wl.n_workers * wbytes * P + (3 << 30)
    free_b, _ = torch.cuda.mem_get_info(dev)
    if need > free_b:
        raise RuntimeError(f"needs {need / 1e9:.0f} GB of device memory, {free_b / 1e9:.0f} GB free")
    events = wl.trace()
    dg = DeviceGenerator(lay, wl.seed, device=dev)
    bufs = [torch.empty(P, dtype=wdt, device=dev) for _ in range(wl.n_workers)]
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)
    out = {"workload": f"{wl.name}: P={P}, {wl.n_workers} workers / {wl.n_lps} LPS, {('f32', 'bf16')[wl.worker_dtype]} copies, "
                       f"whole trace of {len(events)} events", "l2": "256 MB written after each generated input"}
    for label, mb in (("per_event", 1), ("fused", args.max_batch)):
        h = hb.Halos(dg.theta_init(), wl.worker_lps, lay.numel, worker_dtype=wl.worker_dtype, chunk_elems=args.chunk_elems, **wl.hyper())

        def producer(index, worker, rnd):
            r = dg.worker_result(h.peek(hb.BUF_THETA0, worker), worker, rnd, out=bufs[worker], worker_dtype=wl.worker_dtype)
            flush.zero_()
            return r
        h.replay(events[:64], producer, want_log=False, max_batch=mb)        # warm-up
        h.timing_enable(True)
        h.replay(events[64:], producer, want_log=False, max_batch=mb)
        rec = h.timing_launches()
        h.close()
        table = kernel_table(rec, P)
        for k in table.values():
            if k["GBps"]:
                k["frac_of_measured"] = k["GBps"] / peak
                k["frac_of_8TBps"] = k["GBps"] / 8000.0
        kernel_s = float(rec["ms"].astype(np.float64).sum()) * 1e-3
        out[label] = {"kernels": {k: v for k, v in table.items() if v["launches"]},
                      "params_per_s_kernel_time": float(rec["events"].sum()) * P / kernel_s}
        del h
    del bufs, flush
    return out


def run_kernel_table(args):
    """CUDA-event GB/s of EVERY kernel of the library, including those the trace-driven runs rarely or never use
    (standalone push, delayed-Nesterov plain/refresh, materialised deltas, every batch size 2..8, GPS+merge), on a
    small-memory case: the 70M layout, 8 workers on one LPS, both worker dtypes.  Every buffer is larger than L2."""
    import torch
    from paper_2506_04531_b200 import binding as hb, build as _build
    from paper_2506_04531_b200.inputs import gen, layouts, trace as tr
    _build.build()
    dev = torch.device("cuda", 0)
    peak, peak_kind = measured_peak_gbs()
    lay = layouts.named_layout("70m")
    P = lay.P
    rows = []

    def add(label, wname, rec):
        for k, name in enumerate(hb.KERNEL_NAMES):
            r = rec[rec["kind"] == k]
            for bpp in sorted(set(r["bytes_per_param"].tolist())):
                q = r[r["bytes_per_param"] == bpp]
                for nev in sorted(set(q["events"].tolist())):
                    z = q[q["events"] == nev]
                    ms = float(z["ms"].astype(np.float64).mean())
                    gbps = bpp * P / 1e9 / (ms * 1e-3)
                    rows.append({"case": label, "worker_dtype": wname, "kernel": name, "events_per_launch": int(nev),
                                 "bytes_per_param": int(bpp), "launches": int(len(z)), "mean_us": ms * 1e3, "GBps": gbps,
                                 "frac_of_measured": gbps / peak, "frac_of_8TBps": gbps / 8000.0})

    for wdt, wname in ((gen.F32, "f32"), (gen.BF16, "bf16")):
        tdt = torch.float32 if wdt == gen.F32 else torch.int16
        init = torch.randn(P, device=dev) * 0.02
        res = []
        for w in range(8):
            t = init + 1e-3 * torch.randn(P, device=dev)
            res.append(t if wdt == gen.F32 else t.to(torch.bfloat16).view(torch.int16))
        for label, kw in (("paper rule", {}),
                          ("delayed Nesterov d_l=3 d_g=2", dict(optimizer=hb.OPT_DELAYED_NESTEROV, delay_l=3, delay_g=2, eta_l=0.6, eta_g=0.3)),
                          ("materialised delta", dict(flags=hb.FLAG_MATERIALISE_DELTA)),
                          ("statistics on", dict(flags=hb.FLAG_STATS))):
            if "materialised" in label and kw.get("optimizer"):
                continue
            h = hb.Halos(init, [0] * 8, lay.numel, worker_dtype=wdt, K=1 << 20, **kw)
            ev1 = np.zeros(1, dtype=tr.EVENT_DTYPE)

            def calls():
                # call by call: arrive, standalone push, GPS, merge, and the fused GPS+merge
                for w in range(4):
                    h.worker_delta(w, res[w])
                    h.lps_apply(0, w)
                h.lps_push(0); h.gps_merge(0); h.lps_pull(0)
                h.lps_push(0); h.gps_merge_pull(0)
                if "materialised" in label:
                    return
                # fused arrivals: batches of every size 2..8 (distinct workers), without and with a push
                for nb in range(2, 9):
                    ev = np.zeros(nb, dtype=tr.EVENT_DTYPE)
                    ev["worker"] = np.arange(nb)
                    h.replay(ev, lambda i, w, r: res[w], want_log=False, max_batch=nb)
            calls()
            torch.cuda.synchronize(dev)
            h.timing_enable(True)
            for _ in range(6):
                calls()
            add(label, wname, h.timing_launches())
            h.close()
        # pushes fused into the launch that closes a window: K = 1 (single arrival) and K = 4 (batch of four)
        for Kw in (1, 4):
            h = hb.Halos(init, [0] * 8, lay.numel, worker_dtype=wdt, K=Kw)
            ev = np.zeros(Kw, dtype=tr.EVENT_DTYPE)
            ev["worker"] = np.arange(Kw)
            for rep in range(7):
                if rep == 1:
                    h.timing_enable(True)
                h.replay(ev, lambda i, w, r: res[w], want_log=False, max_batch=Kw)
                h.gps_merge_pull(0)
            add(f"K={Kw} (Delta formed by the launch that closes the window)", wname, h.timing_launches())
            h.close()
        del res, init
        torch.cuda.empty_cache()
    print(json.dumps({"kernel_table": rows, "P": P, "peak_GBps": peak, "peak_source": peak_kind}))
    return 0


# ------------------------------------------------------------------------------------ shared by both arms
DEVICE_BUDGET_BYTES = 160 << 30     # of a B200's 180 GB: the context's state plus the resident worker results of the timed steps


def events_per_step(wl, steps: int, asked: int) -> int:
    """Step length: 128 events unless asked otherwise, cut down so that the state and the results of all timed
    steps fit the device budget (~96% of the events are arrivals).  A function of the arguments only, so that
    both arms of the benchmark replay the same windows."""
    wbytes = 4 if wl.worker_dtype == 0 else 2
    P = wl.layout.P
    state = (2 + 5 * wl.n_lps + (1 + wl.n_lps if wl.optimizer else 0)) * 4 * P + wl.n_workers * wbytes * P
    fit = max(1, (DEVICE_BUDGET_BYTES - state) // (wbytes * P))
    eps = asked if asked > 0 else 128
    return int(max(1, min(eps, (fit * 100 // 96) // max(1, steps))))


def spread(xs):
    xs = [float(x) for x in xs]
    return {"median": float(np.median(xs)), "min": min(xs), "max": max(xs), "n": len(xs),
            "rel_spread": (max(xs) - min(xs)) / float(np.median(xs)) if xs and np.median(xs) else None}


def kernel_table(records, P: int, elapsed_ms=None):
    """Per kernel kind, from the library's per-launch records: launches, events carried out, mean duration and
    achieved GB/s on the algorithmic bytes the library accounts for each launch."""
    from paper_2506_04531_b200 import binding as hb
    out = {}
    for k, name in enumerate(hb.KERNEL_NAMES):
        r = records[records["kind"] == k]
        n = int(len(r))
        ms = float(r["ms"].astype(np.float64).sum())
        byts = float((r["bytes_per_param"].astype(np.float64) * P).sum())
        out[name] = {"launches": n, "events": int(r["events"].sum()), "mean_ms": (ms / n if n else None),
                     "bytes_per_param": (byts / P / n if n else None), "GBps": (byts / 1e9 / (ms * 1e-3) if n else None)}
        if elapsed_ms:
            out[name]["share_of_step"] = ms / elapsed_ms
    return out


# ------------------------------------------------------------------------------------ main
def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=10)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="160m", choices=["toy", "70m", "160m", "160m_dn", "410m", "70m_f32_small"])
    ap.add_argument("--events-per-step", type=int, default=0,
                    help="events per step; 0 = 128, reduced so that the results of all timed steps fit in HBM")
    ap.add_argument("--repeats", type=int, default=5, help="how often each timed region is run (state rebuilt untimed in between)")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-configs", action="store_true", help="skip the per-kernel tables of the other configurations")
    ap.add_argument("--cpu-budget-s", type=float, default=15.0)
    ap.add_argument("--chunk-elems", type=int, default=0)
    ap.add_argument("--max-batch", type=int, default=8,
                    help="multi-event fusion in the driver: up to this many arrivals per launch (1 = one kernel per event)")
    ap.add_argument("--launch-log", default="", help="write one record per timed launch of the reported run (.jsonl or .csv)")
    ap.add_argument("--sweep", action="store_true", help="bandwidth sweep over buffer sizes instead of the default line")
    ap.add_argument("--sweep-max", type=int, default=0, help="largest size to include (0 = all)")
    ap.add_argument("--kernel-table", action="store_true", help="CUDA-event GB/s of every kernel of the library on a 70M-size layout")
    ap.add_argument("--cpu-table", action="store_true", help="oracle rates per event kind for every configuration (CPU only)")
    args = ap.parse_args()
    if args.sweep:
        return run_sweep(args)
    if args.kernel_table:
        return run_kernel_table(args)
    if args.cpu_table:
        return run_cpu_table(args)
    if args.warmup < 3 and args.impl == "ours":
        args.warmup = 3

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))

    from paper_2506_04531_b200.inputs import workloads
    wl = workloads.workload(args.workload)
    lay = wl.layout
    P = lay.P
    wname = {0: "f32", 1: "bf16"}[wl.worker_dtype]
    eps = events_per_step(wl, args.steps, args.events_per_step)
    config = {"workload": f"{wl.name}: decoder layout P={P} ({lay.n_tensors} tensors), {wl.n_workers} workers over "
                          f"{wl.n_lps} LPS, 1 GPS, fp32 master + {wname} worker copies, K={wl.K}, paper hyperparameters",
              "events_per_step": eps, "trace_seed": wl.seed, "max_batch": args.max_batch,
              "l2": "every buffer (%.0f MB) is larger than L2; no flush needed" % (P * 4 / 1e6),
              "parallelism": "index-sharded replicas, no collective" if world > 1 else "single GPU"}

    # ---------------------------------------------------------------- reference arm = the oracle
    if args.impl == "reference":
        if rank != 0:
            return 0
        events = window_events(args.steps + args.warmup, eps, wl)
        # every step replays its whole window (the state carries over), on an index slice small enough
        # for the run to end within a few minutes
        S = min(1 << 22, P)
        rep = OracleReplayer(wl, S)
        t_total, total_done = 0.0, 0
        for s in range(args.steps + args.warmup):
            win = events[s * eps:(s + 1) * eps]
            spent, done = rep.run(win)
            if s >= args.warmup:
                t_total += spent
                total_done += done
        rep.close()
        value = total_done * S / t_total
        line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
                "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * t_total / max(1, args.steps),
                "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32",
                "data": "synthetic", "config": config,
                "cpu_baseline": {"value": value, "unit": UNIT, "cores": 1, "kind": "oracle",
                                 "sample": f"every step's {eps} events on the index slice [0,{S}) of {P} parameters"},
                "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
                "gpu_launches": 0}
        print(json.dumps(line))
        return 0

    # ---------------------------------------------------------------- our arm
    import torch
    import torch.distributed as dist
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the update path has no CPU implementation")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)

    from paper_2506_04531_b200 import binding as hb, build as _build
    if rank == 0:
        _build.build()
    if world > 1:
        dist.barrier()
    from paper_2506_04531_b200.inputs import gen
    from paper_2506_04531_b200.inputs.gen_cuda import DeviceGenerator

    # ------------------------------------------------------------------ inputs of the timed regions
    # A worker's result is theta_H = theta_0 + noise, where theta_0 is the model the LPS last scheduled
    # it: it depends on the state.  (Feeding fixed targets instead turns the asynchronous hierarchy into
    # an unstable control loop and the models overflow within a few thousand events.)  To time with the
    # true values AND with every input resident in HBM, the K timed steps are first executed once,
    # untimed, with the generator in the loop, and every result is kept in its own buffer; the state is
    # then rebuilt (same seed, same warm-up: bit-identical) and the timed runs read the stored results.
    # The number of results that fit in HBM bounds the length of a step.
    wbytes = 4 if wl.worker_dtype == gen.F32 else 2
    wdt = torch.float32 if wl.worker_dtype == gen.F32 else torch.int16
    K, W = args.steps, args.warmup
    events = window_events(W + K, eps, wl)
    from paper_2506_04531_b200.inputs import trace as tr
    timed_events = events[W * eps:(W + K) * eps]
    arrive_slots = {int(i): n for n, i in enumerate(np.nonzero(timed_events["kind"] == tr.ARRIVE)[0])}
    n_timed_arrivals = len(arrive_slots)
    n_state_bufs = 2 + 5 * wl.n_lps + (1 + wl.n_lps if wl.optimizer else 0)
    state_bytes = n_state_bufs * 4 * P + wl.n_workers * wbytes * P
    free_b, total_b = torch.cuda.mem_get_info(dev)
    if (n_timed_arrivals + 3) * wbytes * P + state_bytes + (2 << 30) > free_b:
        raise SystemExit(f"{n_timed_arrivals} resident results do not fit in the {free_b / 1e9:.0f} GB of free device memory")
    config["inputs"] = (f"theta_H = theta_0 + sigma z per arrival (faithful), {n_timed_arrivals} results of the timed steps "
                        f"pre-generated by an untimed pass and resident in HBM ({n_timed_arrivals * wbytes * P / 1e9:.1f} GB)")

    seed = wl.seed + 1000 * rank                      # each rank: its own shard of a larger model
    dgen = DeviceGenerator(lay, seed, device=dev)
    scratch = torch.empty(P, dtype=wdt, device=dev)   # warm-up results (one at a time: max_batch = 1)

    def fresh_context():
        """A context in the state right before the first timed step (deterministic)."""
        init = dgen.theta_init()
        h = hb.Halos(init, wl.worker_lps, lay.numel, worker_dtype=wl.worker_dtype, chunk_elems=args.chunk_elems, **wl.hyper())
        del init

        def gen_into_scratch(index, worker, rnd):
            return dgen.worker_result(h.peek(hb.BUF_THETA0, worker), worker, rnd, out=scratch, worker_dtype=wl.worker_dtype)
        for s in range(W):
            h.replay(events[s * eps:(s + 1) * eps], gen_into_scratch, want_log=False, max_batch=1)
        return h

    def state_digest(h):
        """Order-independent 64-bit checksums of the models (to check that the runs ended in the same state)."""
        out = []
        for which, idx in [(hb.BUF_THETA_G, 0), (hb.BUF_M_G, 0)] + [(hb.BUF_THETA_L, l) for l in range(wl.n_lps)]:
            t = h.peek(which, idx)
            if not bool(torch.isfinite(t).all()):
                raise SystemExit("non-finite model values")
            out.append(int(t.view(torch.int32).to(torch.int64).sum().item()))
        return out

    # ---- untimed pass: generate and keep the results of the K timed steps ----
    resident = torch.empty((n_timed_arrivals, P), dtype=wdt, device=dev)
    h = fresh_context()
    for s in range(K):
        base = s * eps

        def gen_and_keep(index, worker, rnd, base=base):
            return dgen.worker_result(h.peek(hb.BUF_THETA0, worker), worker, rnd, out=resident[arrive_slots[base + index]],
                                      worker_dtype=wl.worker_dtype)
        h.replay(timed_events[base:base + eps], gen_and_keep, want_log=False, max_batch=1)
    want_digest = state_digest(h)
    h.close()
    del h
    torch.cuda.empty_cache()

    peak, peak_kind = measured_peak_gbs()

    # per step: the table of result pointers of its events (the resident results), built once outside the timed regions
    step_tables = [hb.result_table(timed_events[s * eps:(s + 1) * eps],
                                   [resident[arrive_slots[s * eps + k]] if (s * eps + k) in arrive_slots else None for k in range(eps)])
                   for s in range(K)]

    def timed_region(max_batch, instrumented=True):
        """K timed steps from the state after the warm-up, reading the resident results.  instrumented: the library
        brackets every launch with CUDA events (per-kernel durations; costs ~4 us per launch)."""
        h = fresh_context()
        torch.cuda.synchronize(dev)
        h.timing_enable(instrumented)
        launches0 = h.info()["launches"]
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize(dev)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        with ClockSampler(local_rank, period_s=0.01) as clk:
            e0.record()
            for s in range(K):
                base = s * eps
                # the results exist already: table-driven replay (no Python per event).  Streaming form: arrivals still
                # waiting for companions at the end of a step may be fused with arrivals of the next step; everything
                # is launched before the region ends
                h.replay_results(timed_events[base:base + eps], step_tables[s], want_log=False, max_batch=max_batch, keep_queued=True)
            h.flush()
            e1.record()
            torch.cuda.synchronize(dev)
        if world > 1:
            dist.barrier()
        elapsed_ms = e0.elapsed_time(e1)
        launches = h.info()["launches"] - launches0
        records = h.timing_launches()
        h.timing_enable(False)
        if state_digest(h) != want_digest:
            raise SystemExit("the timed run did not end in the state of the generating pass")
        h.close()
        units = float(K * eps) * P
        t_ms, units_all = reduce_over_ranks(dist if world > 1 else None, elapsed_ms, units, dev)
        if not instrumented:
            return {"value": units_all / (t_ms * 1e-3), "ms_per_step": t_ms / K, "launches": int(launches)}
        per_kernel = kernel_table(records, P, elapsed_ms)
        dominant = max(per_kernel, key=lambda k: (per_kernel[k]["share_of_step"] or 0))
        d = per_kernel[dominant]
        d_bytes = d["bytes_per_param"] * P
        traffic = max(0.0, d_bytes - L2_WRITE_RESIDUE_BYTES)    # as ncu measures it (see the comment at L2_WRITE_RESIDUE_BYTES)
        roofline = {"bound": "hbm", "kernel": f"{dominant}_kernel<{wname}>", "achieved": d["GBps"], "peak": peak,
                    "unit": "GB/s", "frac": d["GBps"] / peak, "traffic": traffic,
                    "peak_source": f"of {peak_kind}", "algorithmic_bytes_per_launch": d_bytes, "per_kernel": per_kernel}
        if dominant == "arrive_multi":
            roofline["arrivals_per_multi_launch"] = d["events"] / d["launches"]
        return {"value": units_all / (t_ms * 1e-3), "ms_per_step": t_ms / K, "launches": int(launches),
                "roofline": roofline, "clocks": clk.summary(), "records": records}

    def repeated(max_batch):
        """The region `--repeats` times (state rebuilt, untimed, in between); reports the median run with the spread."""
        runs = [timed_region(max_batch) for _ in range(max(1, args.repeats))]
        runs.sort(key=lambda r: r["value"])
        med = runs[len(runs) // 2]
        med["spread"] = {"value": spread([r["value"] for r in runs]),
                         "dominant_kernel_GBps": spread([r["roofline"]["achieved"] for r in runs])}
        reasons = sorted({x for r in runs for x in r["clocks"]["reasons"]})
        med["clocks"] = dict(med["clocks"], reasons=reasons)
        # the same region without the per-launch events: what the instrumentation costs
        plain = sorted((timed_region(max_batch, instrumented=False) for _ in range(3)), key=lambda r: r["value"])[1]
        med["uninstrumented"] = {"value": plain["value"], "unit": UNIT, "ms_per_step": plain["ms_per_step"],
                                 "note": "same region, per-launch CUDA events off (median of 3)"}
        return med

    per_event = repeated(1)                               # one kernel per event: the per-event figure of the metric
    fused = repeated(args.max_batch) if args.max_batch > 1 else None   # multi-event fusion in the driver
    if args.launch_log and rank == 0:
        from paper_2506_04531_b200 import metrics
        metrics.write_launch_records(args.launch_log, per_event["records"], P)

    # ---- end to end: the same steps with the results in pinned HOST memory and every arrival's answer
    # (the model the worker restarts from, Alg. 1 line 12) copied back to pinned host memory ----
    e2e = None
    if not args.no_e2e:
        e2e = run_e2e(args, wl, hb, tr, torch, dist if world > 1 else None, dev, fresh_context, timed_events, arrive_slots,
                      resident, eps, K, P, wbytes, wdt)

    del resident, scratch
    torch.cuda.empty_cache()

    # ---- the other configurations: per-kernel figures over their whole traces (rank 0, N = 1 only) ----
    configs = None
    if rank == 0 and world == 1 and not args.no_configs:
        configs = {}
        for name in ("410m", "70m"):
            if name == wl.name:
                continue
            try:
                configs[name] = config_kernel_table(name, args, torch, dev, peak)
            except Exception as e:              # e.g. not enough free memory for the 410M configuration
                configs[name] = {"error": str(e)[:300]}
            torch.cuda.empty_cache()

    # ---- CPU oracle beside it (rank 0, N = 1 only) ----
    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        cpu_events = wl.trace()                     # the whole configured trace: the sample stops at the time budget
        rate, desc, spent, done, per_kind = oracle_sample(wl, cpu_events, 1 << 22, args.cpu_budget_s, want_kinds=True)
        cpu = {"value": rate, "unit": UNIT, "cores": 1, "kind": "oracle", "sample": desc + f" ({spent:.1f} s)",
               "per_event_kind": per_kind}
        try:
            all_rate, n_cores = oracle_sample_all_cores(wl, cpu_events, 1 << 20, min(6.0, args.cpu_budget_s))
            cpu["all_cores"] = {"value": all_rate, "cores": n_cores,
                                "sample": "one replayer per core, each on its own 1M-parameter slice, up to 6 s"}
        except Exception as e:       # the single-core figure is the baseline; this one is additional context
            cpu["all_cores"] = {"error": str(e)[:200]}

    if rank == 0:
        def public(r):
            return {k: v for k, v in r.items() if k != "records"}
        line = {"metric": METRIC, "value": per_event["value"], "unit": UNIT, "n_gpus": world, "steps": args.steps,
                "warmup": args.warmup, "ms_per_step": per_event["ms_per_step"], "higher_is_better": True, "scaling": "weak",
                "vs_baseline": None, "dtype": "f32", "data": "synthetic", "config": config,
                "clocks": per_event["clocks"], "e2e": e2e, "gpu_launches": per_event["launches"],
                "roofline": per_event["roofline"], "spread": per_event["spread"], "uninstrumented": per_event["uninstrumented"],
                "cpu_baseline": cpu,
                "note": "value = one kernel launch per event (the per-event figure of the metric); fused_replay = the same "
                        "events through the driver's multi-event fusion (bit-identical state, fewer bytes per event)"}
        if fused is not None:
            line["fused_replay"] = {"value": fused["value"], "unit": UNIT, "ms_per_step": fused["ms_per_step"],
                                    "gpu_launches": fused["launches"], "roofline": fused["roofline"], "spread": fused["spread"],
                                    "uninstrumented": fused["uninstrumented"], "clocks": fused["clocks"]}
        if configs is not None:
            line["configs"] = configs
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()
    return 0


if __name__ == "__main__":
    sys.exit(main())
