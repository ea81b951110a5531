"""GPU tests of the fused GPS+merge launch, of the norm statistics inside every fast path, and of the
CUDA path replayed on index shards.  Everything goes through the C ABI binding; expected values come
from the CPU oracle (or from the unfused CUDA replay where the claim is "same bits as unfused")."""
from __future__ import annotations

import numpy as np
import pytest
import torch

from oracle import HalosOracle
from paper_2506_04531_b200 import binding as hb
from paper_2506_04531_b200.inputs import gen, layouts, trace as tr, workloads
from paper_2506_04531_b200.inputs.gen_cuda import DeviceGenerator
from parity_harness import FULL_TRACE_TOL, Lockstep

pytestmark = pytest.mark.gpu

PAPER_HP = dict(eta_l=0.2, beta_l=0.9, eta_g=0.15, beta_g=0.5, alpha=0.25)
DN_HP = dict(eta_l=3.2, beta_l=0.9, eta_g=0.3, beta_g=0.5, alpha=0.25, optimizer=hb.OPT_DELAYED_NESTEROV, delay_l=16, delay_g=2)
STATS_RTOL = 2e-6
ALL_BUFS = list(range(8))


@pytest.fixture(scope="module", autouse=True)
def _built():
    from paper_2506_04531_b200 import build
    build.build()


def _n_of(which, n_workers, n_lps):
    return n_workers if which == hb.BUF_THETA0 else (1 if which in (hb.BUF_THETA_G, hb.BUF_M_G, hb.BUF_ACC_G) else n_lps)


def _same_state(a, b, n_workers, n_lps, bufs=ALL_BUFS):
    for which in bufs:
        for idx in range(_n_of(which, n_workers, n_lps)):
            assert np.array_equal(a.read(which, idx).view(np.uint8), b.read(which, idx).view(np.uint8)), (which, idx)


def _producer(h, dg, lay, worker_lps, wdt=gen.F32):
    tdt = torch.float32 if wdt == gen.F32 else torch.int16
    bufs = [torch.empty(lay.P, dtype=tdt, device="cuda") for _ in worker_lps]
    return lambda index, worker, rnd: dg.worker_result(h.peek(hb.BUF_THETA0, worker), worker, rnd, out=bufs[worker],
                                                       worker_dtype=wdt)


# ---------------------------------------------------------------------------------------------
# GPS update + merge as one launch (Alg. 1 lines 2-4 directly followed by 17-20)
# ---------------------------------------------------------------------------------------------
@pytest.mark.parametrize("hp", [PAPER_HP, DN_HP], ids=["paper_rule", "delayed_nesterov"])
def test_gps_merge_pull_call_matches_oracle(hp):
    lay = layouts.ragged_layout("r", [4099, 33, 20001, 5, 8192, 8191, 3])
    worker_lps = [0, 0, 1]
    hyper = dict(hp, K=2)
    ls = Lockstep(lay, worker_lps, hyper, gen.F32, seed=5, chunk_elems=1024, flags=hb.FLAG_GUARD)
    o, h = ls.o, ls.h
    arrive = np.zeros(1, dtype=tr.EVENT_DTYPE)
    n_round_trips = 0
    for n in range(14):                      # 14 arrivals: windows of 2 close alternately at the two LPSs
        w = [0, 2, 1, 2][n % 4]
        arrive["lps"], arrive["worker"] = worker_lps[w], w
        rec = ls.step(arrive[0])
        if rec["pushed"]:
            l = worker_lps[w]
            h.gps_merge_pull(l)              # CUDA: one launch
            o.gps_recv(l)                    # oracle: the two steps of Algorithm 1
            o.pull(l)
            assert h.counters(l) == o.counters(l)
            n_round_trips += 1
            ls.compare(ls.all_buffers(), FULL_TRACE_TOL)
    assert n_round_trips >= 5 and ls.bit_identical
    assert h.check_guards() == -1
    with pytest.raises(hb.HalosError) as e:  # nothing in flight
        h.gps_merge_pull(0)
    assert e.value.status == hb.ERR_BAD_STATE
    ls.close()


@pytest.mark.parametrize("wdt", [gen.F32, gen.BF16])
def test_driver_fuses_adjacent_gps_and_pull(wdt):
    """On a trace whose LPS 0 sits on the fast link (its PULL follows its GPS_RECV directly) the batched driver
    uses the fused launch; state and log equal the per-event replay, which equals the oracle."""
    wl = workloads.workload("70m")
    lay = layouts.ragged_layout("r", [4099, 33, 20001, 5, 8192, 8191, 3])
    worker_lps = wl.worker_lps
    hp = dict(PAPER_HP, K=6)
    # the trace of the 70M configuration (timing model of its cluster), shortened windows
    events = tr.generate_trace(tr.TraceSpec(P=wl.layout.P, worker_lps=worker_lps, speeds=wl.speeds,
                                            t_profiled_ms=wl.t_profiled_ms, n_arrivals=260, K=6))
    kinds = events["kind"]
    adjacent = sum(1 for k in range(len(events) - 1) if kinds[k] == tr.GPS_RECV and kinds[k + 1] == tr.PULL
                   and events["lps"][k] == events["lps"][k + 1])
    assert adjacent >= 5
    dg = DeviceGenerator(lay, 37)
    ref = hb.Halos(dg.theta_init(), worker_lps, lay.numel, worker_dtype=wdt, chunk_elems=1024, **hp)
    log_ref = ref.replay(events, _producer(ref, dg, lay, worker_lps, wdt))
    fus = hb.Halos(dg.theta_init(), worker_lps, lay.numel, worker_dtype=wdt, chunk_elems=1024, **hp)
    fus.timing_enable(True)
    log_fus = fus.replay(events, _producer(fus, dg, lay, worker_lps, wdt), max_batch=8)
    timing = fus.timing_read()
    assert timing["gps_pull"][0] == adjacent
    assert timing["gps"][0] == int((kinds == tr.GPS_RECV).sum()) - adjacent
    assert timing["pull"][0] == int((kinds == tr.PULL).sum()) - adjacent
    _same_state(ref, fus, len(worker_lps), 2)
    for f in ("index", "kind", "lps", "worker", "t", "t_last", "gps_iter", "worker_staleness", "gps_lag", "pushed"):
        assert np.array_equal(log_ref[f], log_fus[f]), f
    # streaming form with calls cut between a GPS_RECV and its PULL: falls back to the two launches, same state
    cut = hb.Halos(dg.theta_init(), worker_lps, lay.numel, worker_dtype=wdt, chunk_elems=1024, **hp)
    prod = _producer(cut, dg, lay, worker_lps, wdt)
    first = next(k for k in range(len(events) - 1) if kinds[k] == tr.GPS_RECV and kinds[k + 1] == tr.PULL)
    cut.replay(events[:first + 1], prod, max_batch=8, keep_queued=True)
    cut.replay(events[first + 1:], prod, max_batch=8, keep_queued=True)
    cut.flush()
    _same_state(ref, cut, len(worker_lps), 2)
    # ... and the per-event replay equals the oracle on this trace
    o = HalosOracle(gen.theta_init(lay, 37), worker_lps, worker_dtype=wdt, **hp)
    for ev in events:
        kind, l, w = int(ev["kind"]), int(ev["lps"]), int(ev["worker"])
        if kind == tr.ARRIVE:
            o.arrive(w, gen.worker_result(o.buffer("th0", w), lay, 37, w, o.worker_info(w)["round"], worker_dtype=wdt))
        elif kind == tr.GPS_RECV:
            o.gps_recv(l)
        else:
            o.pull(l)
    for which, name in ((hb.BUF_THETA_G, "Theta"), (hb.BUF_M_G, "Mg")):
        assert np.array_equal(fus.read(which).view(np.uint32), o.buffer(name).view(np.uint32))
    for l in (0, 1):
        for which, name in ((hb.BUF_THETA_L, "th"), (hb.BUF_M_L, "ml"), (hb.BUF_ANCHOR, "anchor"), (hb.BUF_INBOX, "inbox"),
                            (hb.BUF_OUTBOX, "outbox")):
            assert np.array_equal(fus.read(which, l).view(np.uint32), o.buffer(name, l).view(np.uint32)), (name, l)
    for h in (ref, fus, cut):
        h.close()
    o.close()


# ---------------------------------------------------------------------------------------------
# norm statistics inside the fast paths: fused launches, delayed Nesterov, materialised deltas
# ---------------------------------------------------------------------------------------------
def _oracle_stats_log(lay, worker_lps, hp, events, seed, wdt=gen.F32, sigma_table=None):
    """Per arrival (in trace order): fp64 sums of squares per tensor of delta, theta_t and (if it pushed) Delta."""
    off = lay.offsets.astype(np.int64)
    o = HalosOracle(gen.theta_init(lay, seed), worker_lps, worker_dtype=wdt, **hp)
    out = []
    for ev in events:
        kind, l, w = int(ev["kind"]), int(ev["lps"]), int(ev["worker"])
        if kind == tr.ARRIVE:
            pushed = o.arrive(w, gen.worker_result(o.buffer("th0", w), lay, seed, w, o.worker_info(w)["round"],
                                                   worker_dtype=wdt))
            rec = [o.sq_norms("delta", l, off), o.sq_norms("th", l, off),
                   o.sq_norms("outbox", l, off) if pushed else np.zeros(lay.n_tensors)]
            out.append(np.stack(rec))
        elif kind == tr.GPS_RECV:
            o.gps_recv(l)
        else:
            o.pull(l)
    o.close()
    return np.stack(out)


@pytest.mark.parametrize("mode", ["paper_f32", "paper_bf16", "delayed_nesterov", "pointer_tables"])
def test_statistics_inside_fused_launches(mode):
    lay = layouts.ragged_layout("r", [4099, 33, 20001, 5, 8192, 8191, 3, 60000])
    worker_lps = [0, 0, 0, 0, 0, 0, 0, 0, 1, 1, 1, 2]
    speeds = [1.0, 1.05, 1.1, 1.15, 1.2, 1.25, 1.3, 3.9, 1.1, 1.2, 3.3, 2.0]
    wdt = gen.BF16 if mode == "paper_bf16" else gen.F32
    hp = dict(DN_HP, K=11, delay_l=3) if mode == "delayed_nesterov" else dict(PAPER_HP, K=11)
    events = tr.generate_trace(tr.TraceSpec(P=lay.P, worker_lps=worker_lps, speeds=speeds, t_profiled_ms=1.0,
                                            n_arrivals=200, K=11))
    n_arr = int((events["kind"] == tr.ARRIVE).sum())
    dg = DeviceGenerator(lay, 43)
    tdt = torch.float32 if wdt == gen.F32 else torch.int16

    def run(max_batch):
        h = hb.Halos(dg.theta_init(), worker_lps, lay.numel, worker_dtype=wdt, chunk_elems=2048, flags=hb.FLAG_STATS, **hp)
        log = torch.full((n_arr + 3, 3, lay.n_tensors), -1.0, dtype=torch.float64, device="cuda")
        h.stats_log(log)
        if mode == "pointer_tables":
            # per-tensor result buffers; the odd tensors of workers 4..7 are shifted by one element, so workers
            # differ in which tensors may take the vector path (such arrivals must not share a launch)
            off = lay.offsets.astype(np.int64)
            parts = []
            for w in range(len(worker_lps)):
                row = []
                for k, n in enumerate(lay.numel):
                    pad = 1 if (4 <= w < 8 and k % 2 == 1) else 0
                    row.append(torch.empty(int(n) + pad + 8, dtype=tdt, device="cuda")[pad:pad + int(n)])
                parts.append(row)

            def producer(index, worker, rnd):
                s0 = h.peek(hb.BUF_THETA0, worker)
                for k, part in enumerate(parts[worker]):
                    dg.worker_result(s0[off[k]:off[k + 1]], worker, rnd, out=part, worker_dtype=wdt, lo=int(off[k]))
                return parts[worker]
        else:
            producer = _producer(h, dg, lay, worker_lps, wdt)
        h.replay(events, producer, max_batch=max_batch)
        last = {l: [h.stats(what, l) for what in range(3)] for l in range(3)}
        torch.cuda.synchronize()
        return h, log.cpu().numpy(), last

    ref, log_ref, last_ref = run(1)
    fus, log_fus, last_fus = run(8)
    assert fus.batch_info()["multi_launches"] > 10           # statistics no longer switch fusion off
    _same_state(ref, fus, len(worker_lps), 3, ALL_BUFS + ([hb.BUF_ACC_L, hb.BUF_ACC_G] if mode == "delayed_nesterov" else []))
    # fused = unfused to the last bit of the fp64 sums, record by record
    assert np.array_equal(log_ref.view(np.uint64), log_fus.view(np.uint64))
    assert (log_fus[n_arr:] == -1.0).all() and (log_fus[:n_arr, :2] >= 0).all()
    for l in range(3):
        for what in range(3):
            assert np.array_equal(last_ref[l][what].view(np.uint64), last_fus[l][what].view(np.uint64)), (l, what)
    # ... and both match the oracle's fp64 sums
    want = _oracle_stats_log(lay, worker_lps, hp, events, 43, wdt)
    np.testing.assert_allclose(log_fus[:n_arr], want, rtol=STATS_RTOL, atol=1e-300)
    assert (want[:, 2].sum(axis=1) > 0).sum() >= 10           # pushes happened and were recorded
    ref.close()
    fus.close()


def test_statistics_with_materialised_deltas_and_log_capacity():
    lay = layouts.ragged_layout("r", [4099, 33, 20001, 5, 8192])
    worker_lps = [0, 0, 1]
    hp = dict(PAPER_HP, K=3)
    events = tr.random_trace(worker_lps, 40, 3, seed=9)
    n_arr = int((events["kind"] == tr.ARRIVE).sum())
    dg = DeviceGenerator(lay, 47)
    h = hb.Halos(dg.theta_init(), worker_lps, lay.numel, chunk_elems=1024,
                 flags=hb.FLAG_STATS | hb.FLAG_MATERIALISE_DELTA | hb.FLAG_GUARD, **hp)
    cap = n_arr - 4                                           # too small on purpose: later arrivals are dropped
    log = torch.full((cap + 2, 3, lay.n_tensors), -1.0, dtype=torch.float64, device="cuda")
    h.stats_log(log[:cap])
    h.replay(events, _producer(h, dg, lay, worker_lps), max_batch=8)
    torch.cuda.synchronize()
    got = log.cpu().numpy()
    want = _oracle_stats_log(lay, worker_lps, hp, events, 47)
    np.testing.assert_allclose(got[:cap], want[:cap], rtol=STATS_RTOL, atol=1e-300)
    assert (got[cap:] == -1.0).all() and h.check_guards() == -1
    h.stats_log(None)
    with pytest.raises(hb.HalosError) as e:                   # statistics need the flag
        plain = hb.Halos(dg.theta_init(), worker_lps, lay.numel, **hp)
        plain.stats_log(log)
    assert e.value.status == hb.ERR_BAD_STATE
    plain.close()
    with pytest.raises(hb.HalosError) as e:                   # and chunks the reduction can hold
        hb.Halos(dg.theta_init(), worker_lps, lay.numel, chunk_elems=16384, flags=hb.FLAG_STATS, **hp)
    assert e.value.status == hb.ERR_UNSUPPORTED
    with pytest.raises(hb.HalosError) as e:
        hb.Halos(torch.zeros(8, device="cuda"), [0], flags=hb.FLAG_MATERIALISE_DELTA, **dict(DN_HP))
    assert e.value.status == hb.ERR_UNSUPPORTED
    h.close()


# ---------------------------------------------------------------------------------------------
# index-sharded replicas of the CUDA path: two contexts on the two halves of the parameter range
# reproduce the unsharded context (every step is elementwise, so shards exchange nothing)
# ---------------------------------------------------------------------------------------------
@pytest.mark.parametrize("wdt", [gen.F32, gen.BF16])
def test_cuda_path_on_index_shards_equals_unsharded(wdt):
    lay = layouts.ragged_layout("r", [4099, 33, 20001, 5, 8192, 8191, 3, 30011])
    P = lay.P
    cut = 4099 + 33 + 9000 + 5                 # inside the third tensor, not on a vector or chunk boundary
    off = lay.offsets.astype(np.int64)
    assert cut % 8 != 0 and not (off == cut).any()

    def shard_numel(lo, hi):
        """The layout's tensors clipped to [lo, hi): how a rank derives its own tensor list."""
        return [int(min(hi, off[k + 1]) - max(lo, off[k])) for k in range(lay.n_tensors) if min(hi, off[k + 1]) > max(lo, off[k])]

    worker_lps = [0, 0, 0, 1, 1, 2]
    hp = dict(PAPER_HP, K=5)
    events = tr.generate_trace(tr.TraceSpec(P=P, worker_lps=worker_lps, speeds=[1.0, 1.1, 3.5, 1.3, 2.0, 1.7],
                                            t_profiled_ms=1.0, n_arrivals=150, K=5))
    dg = DeviceGenerator(lay, 53)
    tdt = torch.float32 if wdt == gen.F32 else torch.int16
    full = hb.Halos(dg.theta_init(), worker_lps, lay.numel, worker_dtype=wdt, chunk_elems=1024, **hp)
    log_full = full.replay(events, _producer(full, dg, lay, worker_lps, wdt), max_batch=8)
    shards = []
    for lo, hi in ((0, cut), (cut, P)):
        numel = shard_numel(lo, hi)
        assert sum(numel) == hi - lo
        h = hb.Halos(dg.theta_init(lo, hi), worker_lps, numel, worker_dtype=wdt, chunk_elems=1024, **hp)
        bufs = [torch.empty(hi - lo, dtype=tdt, device="cuda") for _ in worker_lps]

        def producer(index, worker, rnd, h=h, bufs=bufs, lo=lo):
            # the shard's own snapshot, the generator's global index offset: no value comes from the full context
            return dg.worker_result(h.peek(hb.BUF_THETA0, worker), worker, rnd, out=bufs[worker], worker_dtype=wdt, lo=lo)
        log = h.replay(events, producer, max_batch=8)
        for f in ("t", "t_last", "gps_iter", "worker_staleness", "gps_lag", "pushed"):
            assert np.array_equal(log[f], log_full[f]), f
        shards.append(h)
    for which in ALL_BUFS:
        for idx in range(_n_of(which, len(worker_lps), 3)):
            glued = np.concatenate([s.read(which, idx) for s in shards])
            assert np.array_equal(glued.view(np.uint8), full.read(which, idx).view(np.uint8)), (which, idx)
    for h in shards + [full]:
        h.close()


# ---------------------------------------------------------------------------------------------
# the worker's new start model copied to host memory, overlapping later updates
# ---------------------------------------------------------------------------------------------
@pytest.mark.parametrize("wdt", [gen.F32, gen.BF16])
def test_worker_fetch_host_returns_the_scheduled_model(wdt):
    lay = layouts.ragged_layout("r", [300_001, 33, 2_000_003, 5, 65536])
    worker_lps = [0, 0, 1]
    hp = dict(PAPER_HP, K=3)
    events = tr.random_trace(worker_lps, 40, 3, seed=13)
    dg = DeviceGenerator(lay, 59)
    h = hb.Halos(dg.theta_init(), worker_lps, lay.numel, worker_dtype=wdt, **hp)
    o = HalosOracle(gen.theta_init(lay, 59), worker_lps, worker_dtype=wdt, **hp)
    prod = _producer(h, dg, lay, worker_lps, wdt)
    np_dt = np.float32 if wdt == gen.F32 else np.uint16
    t_dt = torch.float32 if wdt == gen.F32 else torch.int16
    outs, wants = [], []
    for n, ev in enumerate(events):
        kind, l, w = int(ev["kind"]), int(ev["lps"]), int(ev["worker"])
        h.replay(events[n:n + 1], prod, max_batch=8, keep_queued=True)    # arrivals may stay queued: fetch launches them
        if kind == tr.ARRIVE:
            o.arrive(w, gen.worker_result(o.buffer("th0", w), lay, 59, w, o.worker_info(w)["round"], worker_dtype=wdt))
            dst = torch.empty(lay.P, dtype=t_dt).pin_memory()
            h.worker_fetch_host(w, dst)          # not waited for: later updates (of this worker too) run on
            outs.append(dst)
            wants.append(o.buffer("th0", w).copy())
        elif kind == tr.GPS_RECV:
            o.gps_recv(l)
        else:
            o.pull(l)
    h.flush()
    h.fetch_sync()
    assert len(outs) >= 25
    for dst, want in zip(outs, wants):
        assert np.array_equal(dst.numpy().view(np_dt), want.view(np_dt))
    h.close()
    o.close()


# ---------------------------------------------------------------------------------------------
# per-launch records: kind, events and the algorithmic bytes the library accounts (bench.py's GB/s rest on them)
# ---------------------------------------------------------------------------------------------
@pytest.mark.parametrize("wdt,wb", [(gen.F32, 4), (gen.BF16, 2)])
def test_launch_records_account_algorithmic_bytes(wdt, wb):
    P = 1 << 16
    init = torch.linspace(-1, 1, P, device="cuda")
    tdt = torch.float32 if wdt == gen.F32 else torch.int16
    res = [torch.zeros(P, dtype=tdt, device="cuda") for _ in range(4)]
    ev = np.zeros(3, dtype=tr.EVENT_DTYPE)
    ev["worker"] = [0, 1, 2]

    def run(h, fused_window):
        h.timing_enable(True)
        h.worker_delta(3, res[3]); h.lps_apply(0, 3)                      # arrive alone
        h.lps_push(0); h.gps_merge(0); h.lps_pull(0)                        # push, GPS, merge
        h.replay(ev, lambda i, w, r: res[w], max_batch=8)                   # three arrivals in one launch
        if fused_window:
            h.gps_merge_pull(0)                                            # (the batch closed the window)
        rec = h.timing_launches()
        return [(hb.KERNEL_NAMES[int(r["kind"])], int(r["events"]), int(r["bytes_per_param"])) for r in rec], rec

    h = hb.Halos(init, [0, 0, 0, 0], worker_dtype=wdt, K=3, **PAPER_HP)     # the merge sets t_last = 1: t = 4 closes the window
    got, rec = run(h, True)
    assert got == [("arrive", 1, 16 + 3 * wb), ("push", 0, 12), ("gps", 1, 24), ("pull", 1, 16),
                   ("arrive_multi", 3, 16 + 9 * wb + 8), ("gps_pull", 2, 36)]
    assert (rec["ms"] > 0).all() and h.timing_read()["arrive_multi"][0] == 1
    h.close()
    # delayed Nesterov, refresh every 2nd LPS update and every 2nd GPS update: +8 bytes where the momentum moves
    h = hb.Halos(init, [0, 0, 0, 0], worker_dtype=wdt, K=3, **dict(DN_HP, delay_l=2, delay_g=2))
    got, _ = run(h, True)
    assert got == [("arrive", 1, 16 + 3 * wb), ("push", 0, 12), ("gps", 1, 24), ("pull", 1, 16),
                   ("arrive_multi", 3, 16 + 9 * wb + 8 + 8), ("gps_pull", 2, 36 + 8)]
    h.close()
    # materialised delta: the arrive reads delta (4 B) instead of theta_H and theta_0
    h = hb.Halos(init, [0, 0, 0, 0], worker_dtype=wdt, K=100, flags=hb.FLAG_MATERIALISE_DELTA, **PAPER_HP)
    got, _ = run(h, False)
    assert got[0] == ("arrive", 1, 20 + wb) and [g[0] for g in got[4:]] == ["arrive"] * 3
    # new entry points refuse bad arguments without touching the state
    for call, status in ((lambda: h.gps_merge_pull(7), hb.ERR_INVALID_ARG), (lambda: h.gps_merge_pull(0), hb.ERR_BAD_STATE),
                         (lambda: h.worker_fetch_host(9, torch.empty(P, dtype=tdt).pin_memory()), hb.ERR_INVALID_ARG)):
        with pytest.raises(hb.HalosError) as e:
            call()
        assert e.value.status == status
    h.close()


# ---------------------------------------------------------------------------------------------
# randomised equivalence: any split into streaming calls, any batch limit, both optimizers and
# worker dtypes -- the fused driver leaves the state and the log of the per-event replay
# ---------------------------------------------------------------------------------------------
@pytest.mark.parametrize("seed", range(8))
def test_fused_driver_equals_per_event_replay_on_random_traces(seed):
    rng = np.random.default_rng(900 + seed)
    n_lps = int(rng.integers(1, 4))
    n_workers = int(rng.integers(n_lps, 11))
    worker_lps = [int(x) for x in np.concatenate([np.arange(n_lps), rng.integers(0, n_lps, n_workers - n_lps)])]
    K = int(rng.integers(1, 7))
    wdt = gen.BF16 if seed % 2 else gen.F32
    dn = seed % 4 >= 2
    hp = dict(DN_HP, K=K, delay_l=int(rng.integers(1, 5)), delay_g=int(rng.integers(1, 4))) if dn else dict(PAPER_HP, K=K)
    sizes = [int(x) for x in rng.integers(1, 9000, size=int(rng.integers(1, 7)))]
    lay = layouts.ragged_layout("r", sizes)
    events = tr.random_trace(worker_lps, 220, K, seed=seed)
    dg = DeviceGenerator(lay, 300 + seed)
    mk = lambda: hb.Halos(dg.theta_init(), worker_lps, lay.numel, worker_dtype=wdt, chunk_elems=int(rng.choice([256, 1024, 4096])),
                          flags=hb.FLAG_GUARD, **hp)
    ref = mk()
    log_ref = ref.replay(events, _producer(ref, dg, lay, worker_lps, wdt))
    fus = mk()
    prod = _producer(fus, dg, lay, worker_lps, wdt)
    logs, pos = [], 0
    while pos < len(events):                     # random call lengths, random batch limits, streaming or flushing calls
        n = int(rng.integers(1, 40))
        logs.append(fus.replay(events[pos:pos + n], prod, max_batch=int(rng.integers(2, 9)), keep_queued=bool(rng.integers(0, 2))))
        pos += n
    fus.flush()
    log_fus = np.concatenate(logs)
    extra = [hb.BUF_ACC_L, hb.BUF_ACC_G] if dn else []
    _same_state(ref, fus, n_workers, n_lps, ALL_BUFS + extra)
    for f in ("kind", "lps", "worker", "t", "t_last", "gps_iter", "worker_staleness", "gps_lag", "pushed"):
        assert np.array_equal(log_ref[f], log_fus[f]), f
    for l in range(n_lps):
        assert ref.counters(l) == fus.counters(l)
    assert fus.check_guards() == -1 and ref.check_guards() == -1
    assert fus.info()["launches"] <= ref.info()["launches"]
    assert int(log_fus["fused"].sum()) > 0
    ref.close()
    fus.close()


# ---------------------------------------------------------------------------------------------
# table-driven replay (results that already exist, no callback) = replay with a producer
# ---------------------------------------------------------------------------------------------
def test_replay_results_equals_replay_with_a_producer():
    lay = layouts.ragged_layout("r", [4099, 33, 20001, 5, 8192])
    worker_lps = [0, 0, 0, 1, 1]
    hp = dict(PAPER_HP, K=4)
    events = tr.random_trace(worker_lps, 120, 4, seed=21)
    dg = DeviceGenerator(lay, 61)
    ref = hb.Halos(dg.theta_init(), worker_lps, lay.numel, chunk_elems=1024, **hp)
    kept = []                                                # every result of the reference run, in event order

    def producer(index, worker, rnd):
        r = dg.worker_result(ref.peek(hb.BUF_THETA0, worker), worker, rnd)
        kept.append((index, r))
        return r
    log_ref = ref.replay(events, producer)
    results = [None] * len(events)
    for index, r in kept:
        results[index] = r
    for mb, streaming in ((1, False), (8, False), (8, True)):
        h = hb.Halos(dg.theta_init(), worker_lps, lay.numel, chunk_elems=1024, **hp)
        if streaming:
            logs = [h.replay_results(events[a:a + 7], results[a:a + 7], max_batch=mb, keep_queued=True) for a in range(0, len(events), 7)]
            h.flush()
            log = np.concatenate(logs)
        else:
            log = h.replay_results(events, hb.result_table(events, results), max_batch=mb)
        _same_state(ref, h, len(worker_lps), 2)
        for f in ("kind", "lps", "worker", "t", "t_last", "gps_iter", "worker_staleness", "gps_lag", "pushed"):
            assert np.array_equal(log_ref[f], log[f]), f
        h.close()
    # an ARRIVE without a result fails that event and leaves nothing registered
    h = hb.Halos(dg.theta_init(), worker_lps, lay.numel, **hp)
    first = int(np.nonzero(events["kind"] == tr.ARRIVE)[0][1])
    broken = list(results)
    broken[first] = None
    with pytest.raises(hb.HalosError) as e:
        h.replay_results(events, broken)
    assert e.value.status == hb.ERR_INVALID_ARG and f"event {first}" in str(e.value)
    assert not h.worker_info(int(events["worker"][first]))["pending"]
    h.close()
    ref.close()
