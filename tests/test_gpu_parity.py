"""Parity of the CUDA library (called through the C ABI) with the CPU oracle on the same seeded
traces and inputs.  Tolerances: max relative error 1e-6 after any single event, 1e-5 after a full
trace (fp32); the arithmetic is mirrored operation by operation, so bit identity is expected and
asserted wherever the whole state is compared."""
from __future__ import annotations

import struct
import zlib
from fractions import Fraction as Fr
from pathlib import Path

import numpy as np
import pytest
import torch

from paper_2506_04531_b200 import binding as hb
from paper_2506_04531_b200.inputs import gen, layouts, trace as tr, workloads
from parity_harness import FULL_TRACE_TOL, PER_EVENT_TOL, Lockstep, default_probes

pytestmark = pytest.mark.gpu

PAPER_HP = dict(eta_l=0.2, beta_l=0.9, eta_g=0.15, beta_g=0.5, alpha=0.25)


@pytest.fixture(scope="module", autouse=True)
def _built():
    from paper_2506_04531_b200 import build
    build.build()


# ---------------------------------------------------------------------------------------------
# the CUDA input generator equals the numpy one bit for bit (they feed the two sides)
# ---------------------------------------------------------------------------------------------
def test_generators_agree():
    from paper_2506_04531_b200.inputs.gen_cuda import DeviceGenerator
    lay = layouts.decoder_layout("tiny", 2, 64, 300)
    dg = DeviceGenerator(lay, 77)
    init = dg.theta_init().cpu().numpy()
    np.testing.assert_array_equal(init.view(np.uint32), gen.theta_init(lay, 77).view(np.uint32))
    np.testing.assert_array_equal(dg.theta_init(1000, 5001).cpu().numpy(), init[1000:5001])
    s0 = torch.from_numpy(init).cuda()
    r = dg.worker_result(s0, 3, 9).cpu().numpy()
    np.testing.assert_array_equal(r.view(np.uint32), gen.worker_result(init, lay, 77, 3, 9).view(np.uint32))
    hb16 = gen.f32_to_bf16_bits(init)
    s0b = torch.from_numpy(hb16.view(np.int16)).cuda()
    rb = dg.worker_result(s0b, 3, 9, worker_dtype=gen.BF16).cpu().numpy().view(np.uint16)
    np.testing.assert_array_equal(rb, gen.worker_result(hb16, lay, 77, 3, 9, worker_dtype=gen.BF16))


# ---------------------------------------------------------------------------------------------
# exact hand expansion on 8 parameters, straight against the golden values
# ---------------------------------------------------------------------------------------------
def test_hand_expansion_on_gpu():
    golden = Path(__file__).parent / "golden" / "hand_expansion_p8.txt"
    rows, bits = [], {}
    for line in golden.read_text().splitlines():
        parts = line.split()
        if not parts or parts[0].startswith("#"):
            continue
        if parts[0] == "bits":
            bits[parts[1]] = [int(x, 16) for x in parts[2:]]
        else:
            rows.append((int(parts[0]), parts[1], [float(Fr(x)) for x in parts[2:]]))
    init = torch.tensor([(j - 4) / 8 for j in range(8)], dtype=torch.float32, device="cuda")
    h = hb.Halos(init, [0, 0, 1], eta_l=0.5, beta_l=0.5, eta_g=0.5, beta_g=0.5, alpha=0.25, K=2)
    which = {"th": hb.BUF_THETA_L, "ml": hb.BUF_M_L, "outbox": hb.BUF_OUTBOX}
    rounds = [0, 0, 0]
    for n, e in enumerate("A0 A2 A1 A0 G0 A2 G1 P0 A1 P1 A0 G0".split(), 1):
        kind, i = e[0], int(e[1])
        if kind == "A":
            s0 = h.read(hb.BUF_THETA0, i)
            noise = np.array([((3 * i + 5 * rounds[i] + 7 * j) % 9 - 4) / 16 for j in range(8)], np.float32)
            rounds[i] += 1
            thH = torch.from_numpy(s0 + noise).cuda()
            h.worker_delta(i, thH)
            if h.lps_apply(int(h.worker_lps[i]), i):
                h.lps_push(int(h.worker_lps[i]))
        elif kind == "G":
            h.gps_merge(i)
        else:
            h.lps_pull(i)
        for ev, name, vals in rows:
            if ev != n:
                continue
            if name == "Theta":
                got = h.read(hb.BUF_THETA_G)
            elif name == "Mg":
                got = h.read(hb.BUF_M_G)
            else:
                got = h.read(which[name[:-1]], int(name[-1]))
            assert got.tolist() == vals, f"event {n} {name}"
    as_bits = lambda a: [struct.unpack("<I", struct.pack("<f", float(x)))[0] for x in a]
    assert as_bits(h.read(hb.BUF_THETA_G)) == bits["Theta"]
    assert as_bits(h.read(hb.BUF_THETA_L, 0)) == bits["th0"]
    assert as_bits(h.read(hb.BUF_THETA_L, 1)) == bits["th1"]
    h.close()


# ---------------------------------------------------------------------------------------------
# tiny and ragged shapes, both worker dtypes, flat and pointer-table inputs, odd chunk sizes
# ---------------------------------------------------------------------------------------------
_SHAPES = {
    "p1": [1], "p3": [3], "p4": [4], "p5": [5], "p8": [8], "p31": [31], "p4097": [4097],
    "ragged": [7, 1, 1024, 3, 513, 2, 4096, 9, 1, 1, 777],
    "ragged_big": [4099, 33, 20001, 5, 8192, 8191],
    "with_empty": [16, 0, 5, 0, 64],
}


@pytest.mark.parametrize("shape", list(_SHAPES))
@pytest.mark.parametrize("wdt", [gen.F32, gen.BF16])
@pytest.mark.parametrize("mode", ["flat", "ptrs", "ptrs_misaligned"])
def test_small_shapes_bit_exact(shape, wdt, mode):
    lay = layouts.ragged_layout(shape, _SHAPES[shape])
    worker_lps = [0, 0, 1, 1, 1]
    events = tr.random_trace(worker_lps, 60, 3, seed=zlib.crc32(f"{shape}/{wdt}/{mode}".encode()) & 0xFFFF)
    chunk = 1024 if shape in ("ragged_big", "p4097") else 0
    ls = Lockstep(lay, worker_lps, dict(K=3, **PAPER_HP), wdt, seed=5, chunk_elems=chunk, input_mode=mode,
                  flags=hb.FLAG_GUARD)
    ls.run(events, check_every=1, full_check_every=20)
    assert ls.bit_identical and ls.max_err == 0.0
    assert ls.h.check_guards() == -1          # no kernel wrote outside its buffers
    ls.close()


@pytest.mark.parametrize("chunk", [8, 64, 1024, 8192, 1 << 20])
def test_chunk_size_invariance(chunk):
    lay = layouts.ragged_layout("r", [4099, 33, 20001, 5, 8192, 8191, 100000])
    worker_lps = [0, 1]
    events = tr.random_trace(worker_lps, 25, 2, seed=9)
    ls = Lockstep(lay, worker_lps, dict(K=2, **PAPER_HP), gen.F32, seed=8, chunk_elems=chunk)
    ls.run(events, check_every=5)
    assert ls.bit_identical
    info = ls.h.info()
    assert info["P"] == lay.P and info["n_tensors"] == lay.n_tensors
    ls.close()


# ---------------------------------------------------------------------------------------------
# configuration 1 ("toy"): 1,048,576 parameters, 4 workers, 2 LPS, 200 arrivals, every event checked
# ---------------------------------------------------------------------------------------------
@pytest.mark.parametrize("name", ["toy", "toy_k4", "paper_cluster_small", "hetero_grouping_small"])
def test_toy_config_every_event(name):
    wl = workloads.workload(name)
    ls = Lockstep(wl.layout, wl.worker_lps, wl.hyper(), wl.worker_dtype, wl.seed)
    ls.run(wl.trace(), check_every=1, full_check_every=50)
    assert ls.bit_identical and ls.max_err <= PER_EVENT_TOL
    # the trace exercised the whole hierarchy
    kinds = [r["kind"] for r in ls.log]
    assert kinds.count(tr.GPS_RECV) >= (4 if name == "toy" else 20)
    assert max(r.get("worker_staleness", 0) for r in ls.log) >= 1
    ls.close()


# ---------------------------------------------------------------------------------------------
# the event-queue driver: same bits as the call-by-call sequence, and the same event log
# ---------------------------------------------------------------------------------------------
@pytest.mark.parametrize("wdt", [gen.F32, gen.BF16])
def test_replay_driver_matches_calls_and_oracle_log(wdt):
    from paper_2506_04531_b200.inputs.gen_cuda import DeviceGenerator
    lay = layouts.decoder_layout("tiny", 2, 64, 300)
    worker_lps = [0, 0, 1, 1]
    hp = dict(K=4, **PAPER_HP)
    events = tr.generate_trace(tr.TraceSpec(P=lay.P, worker_lps=worker_lps, speeds=[1.0, 2.5, 3.0, 1.7],
                                            t_profiled_ms=1.0, n_arrivals=120, K=4))
    ls = Lockstep(lay, worker_lps, hp, wdt, seed=21)
    ls.run(events, check_every=0)
    assert ls.bit_identical

    dg = DeviceGenerator(lay, 21)
    h2 = hb.Halos(dg.theta_init(), worker_lps, lay.numel, worker_dtype=wdt, **hp)
    scratch = torch.empty(lay.P, dtype=torch.float32 if wdt == gen.F32 else torch.int16, device="cuda")

    def producer(index, worker, rnd):
        return dg.worker_result(h2.peek(hb.BUF_THETA0, worker), worker, rnd, out=scratch, worker_dtype=wdt)

    log = h2.replay(events, producer)
    for name, idx in ls.all_buffers():
        a = ls.gpu_values(name, idx)
        which = {"Theta": hb.BUF_THETA_G, "Mg": hb.BUF_M_G, "th": hb.BUF_THETA_L, "ml": hb.BUF_M_L,
                 "anchor": hb.BUF_ANCHOR, "outbox": hb.BUF_OUTBOX, "inbox": hb.BUF_INBOX, "th0": hb.BUF_THETA0}[name]
        b = h2.read(which, idx)
        assert np.array_equal(a.view(np.uint8), b.view(np.uint8)), (name, idx)
    assert len(log) == len(ls.log)
    for rec, want in zip(log, ls.log):
        assert (int(rec["kind"]), int(rec["lps"]), int(rec["t"]), int(rec["t_last"]), int(rec["gps_iter"])) == \
               (want["kind"], want["lps"], want["t"], want["t_last"], want["gps_iter"])
        if want["kind"] == tr.ARRIVE:
            assert int(rec["worker"]) == want["worker"]
            assert int(rec["worker_staleness"]) == want["worker_staleness"]
            assert bool(rec["pushed"]) == want["pushed"]
        if want["kind"] == tr.PULL:
            assert int(rec["gps_lag"]) == want["gps_lag"]
    assert int(log["pushed"].sum()) == int((events["kind"] == tr.GPS_RECV).sum())
    h2.close()
    ls.close()


# ---------------------------------------------------------------------------------------------
# call-order errors leave the state untouched
# ---------------------------------------------------------------------------------------------
def test_state_machine_errors():
    P = 1000
    init = torch.linspace(-1, 1, P, device="cuda")
    h = hb.Halos(init, [0, 1], K=1, **PAPER_HP)
    snap = lambda: [h.read(b, i).copy() for b in (hb.BUF_THETA_L, hb.BUF_M_L, hb.BUF_ANCHOR) for i in (0, 1)] + \
                   [h.read(hb.BUF_THETA_G), h.read(hb.BUF_M_G)]
    before, c_before = snap(), h.counters(0)
    thH = init + 0.01

    def expect(status, fn, *a):
        with pytest.raises(hb.HalosError) as e:
            fn(*a)
        assert e.value.status == status

    expect(hb.ERR_BAD_STATE, h.lps_apply, 0, 0)          # no pending result
    expect(hb.ERR_BAD_STATE, h.gps_merge, 0)             # nothing pushed
    expect(hb.ERR_BAD_STATE, h.lps_pull, 0)              # nothing answered
    expect(hb.ERR_INVALID_ARG, h.lps_apply, 7, 0)
    expect(hb.ERR_INVALID_ARG, h.worker_delta, 9, thH)
    h.worker_delta(0, thH)
    expect(hb.ERR_BAD_STATE, h.worker_delta, 0, thH)     # already pending
    expect(hb.ERR_INVALID_ARG, h.lps_apply, 1, 0)        # worker 0 belongs to LPS 0
    for a, b in zip(before, snap()):
        np.testing.assert_array_equal(a, b)
    assert h.counters(0) == c_before
    assert h.lps_apply(0, 0) is True                     # K = 1: push due
    h.lps_push(0)
    expect(hb.ERR_BAD_STATE, h.lps_push, 0)              # second push while in flight
    expect(hb.ERR_BAD_STATE, h.lps_pull, 0)
    h.gps_merge(0)
    expect(hb.ERR_BAD_STATE, h.gps_merge, 0)
    h.lps_pull(0)
    c = h.counters(0)
    assert (c["t"], c["t_last"], c["phase"], c["i"]) == (1, 1, hb.IDLE, 1)
    expect(hb.ERR_INVALID_ARG, h.read, hb.BUF_THETA_L, 0, P - 1, 5)
    h.close()
    with pytest.raises(ValueError):
        hb.Halos(init, [0], tensor_numel=[3, 4])


# ---------------------------------------------------------------------------------------------
# host-resident worker results (staged copy) give the same bits as device-resident ones
# ---------------------------------------------------------------------------------------------
def test_host_inputs_match_device_inputs():
    lay = layouts.flat_layout("x", 300_001)
    init = torch.from_numpy(gen.theta_init(lay, 4)).cuda()
    a = hb.Halos(init, [0, 0, 0], **PAPER_HP)
    b = hb.Halos(init, [0, 0, 0], **PAPER_HP)
    pinned = [torch.empty(lay.P, dtype=torch.float32).pin_memory() for _ in range(3)]
    for rnd in range(3):
        # two staging buffers: at most two host results may wait for their apply
        for group in ((2, 0), (1,)):
            for w in group:
                res = gen.worker_result(a.read(hb.BUF_THETA0, w), lay, 4, w, rnd)
                pinned[w].copy_(torch.from_numpy(res))
                b.worker_delta_host(w, pinned[w])
                a.worker_delta(w, torch.from_numpy(res).cuda())
            for w in group:
                a.lps_apply(0, w)
                b.lps_apply(0, w)
        np.testing.assert_array_equal(a.read(hb.BUF_THETA_L, 0), b.read(hb.BUF_THETA_L, 0))
        np.testing.assert_array_equal(a.read(hb.BUF_THETA0, 1), b.read(hb.BUF_THETA0, 1))
    for w in (0, 1):
        b.worker_delta_host(w, pinned[w])
    with pytest.raises(hb.HalosError) as e:
        b.worker_delta_host(2, pinned[2])          # both staging buffers are taken
    assert e.value.status == hb.ERR_BAD_STATE
    a.close()
    b.close()


# ---------------------------------------------------------------------------------------------
# optional per-tensor squared norms
# ---------------------------------------------------------------------------------------------
def test_norm_statistics():
    lay = layouts.ragged_layout("r", [4099, 33, 20001, 5, 8192, 100000])
    worker_lps = [0, 1]
    ls = Lockstep(lay, worker_lps, dict(K=2, **PAPER_HP), gen.F32, seed=3, flags=hb.FLAG_STATS, chunk_elems=2048)
    events = tr.random_trace(worker_lps, 12, 2, seed=1)
    off = lay.offsets.astype(np.int64)
    for ev in events:
        rec = ls.step(ev)
        if rec["kind"] == tr.ARRIVE:
            np.testing.assert_allclose(ls.h.stats(0, rec["lps"]), ls.o.sq_norms("delta", rec["lps"], off), rtol=2e-6)
            np.testing.assert_allclose(ls.h.stats(2, rec["lps"]), ls.o.sq_norms("th", rec["lps"], off), rtol=2e-6)
            if rec["pushed"]:
                np.testing.assert_allclose(ls.h.stats(1, rec["lps"]), ls.o.sq_norms("outbox", rec["lps"], off), rtol=2e-6)
    ls.compare(ls.all_buffers(), FULL_TRACE_TOL)
    assert ls.bit_identical
    ls.close()


# ---------------------------------------------------------------------------------------------
# LLM-shaped configurations at full size on the GPU; the oracle replays probe windows
# ---------------------------------------------------------------------------------------------
def _run_config(name, n_events, check_every, full_every):
    """Lock-step, call by call, with the oracle on the probe set: the first and last 64K elements, 8K around
    every tensor boundary and 16 random windows of 64K; the written buffers are compared after every
    check_every-th event at the per-event tolerance, all buffers every full_every events and at the end."""
    wl = workloads.workload(name)
    probes = default_probes(wl.layout, seed=wl.seed)
    off = wl.layout.offsets.astype(np.int64)
    assert all(any(lo < b < hi for lo, hi in probes) for b in off[1:-1])      # every tensor boundary is inside a window
    ls = Lockstep(wl.layout, wl.worker_lps, wl.hyper(), wl.worker_dtype, wl.seed, probes=probes)
    events = wl.trace()[:n_events]
    ls.run(events, check_every=check_every, full_check_every=full_every)
    assert ls.max_err <= FULL_TRACE_TOL
    assert ls.bit_identical
    kinds = [r["kind"] for r in ls.log]
    assert kinds.count(tr.PULL) >= 2
    ls.close()
    return ls


def test_config_70m_bf16_full_trace():
    _run_config("70m", None, check_every=1, full_every=250)


def test_config_160m_fp32_full_trace():
    _run_config("160m", None, check_every=1, full_every=500)


def test_config_410m_fp32_staleness_order():
    # 32 workers with fp32 copies: ~89 GB on the device
    torch.cuda.empty_cache()
    free, _ = torch.cuda.mem_get_info()
    if free < 100 * (1 << 30):
        pytest.skip("needs ~95 GB of free device memory")
    ls = _run_config("410m", 700, check_every=2, full_every=0)   # 700 events: every LPS, the slow region's too, has merged
    # the slowed-down region sees the stalest workers' results least often but every LPS made round trips
    by_lps = {}
    for r in ls.log:
        if r["kind"] == tr.PULL:
            by_lps[r["lps"]] = by_lps.get(r["lps"], 0) + 1
    assert set(by_lps) == {0, 1, 2, 3}


# ---------------------------------------------------------------------------------------------
# bandwidth-sweep shapes: flat buffers and the 1.4B-class layout (the largest size), one pass of
# every kernel, sampled outputs against the oracle
# ---------------------------------------------------------------------------------------------
@pytest.mark.parametrize("case,wdt", [("flat_2^24", gen.F32), ("flat_2^26", gen.BF16), ("decoder_1p4b", gen.F32)])
def test_sweep_shapes_one_pass(case, wdt):
    if case == "decoder_1p4b":
        torch.cuda.empty_cache()
        free, _ = torch.cuda.mem_get_info()
        if free < 70 * (1 << 30):
            pytest.skip("needs ~60 GB of free device memory")
        lay = layouts.named_layout("1p4b")
    else:
        lay = layouts.flat_layout(case, 1 << int(case.split("^")[1]))
    probes = default_probes(lay, width=8192, n_random=12, seed=1)
    ls = Lockstep(lay, [0], dict(K=2, **PAPER_HP), wdt, seed=31, probes=probes)
    ev = np.zeros(7, dtype=tr.EVENT_DTYPE)
    ev["kind"] = [tr.ARRIVE, tr.ARRIVE, tr.GPS_RECV, tr.ARRIVE, tr.PULL, tr.ARRIVE, tr.ARRIVE]
    ls.run(ev, check_every=1)
    assert ls.bit_identical
    assert ls.h.counters(0) == {"t": 5, "t_last": 3, "phase": hb.PUSHED, "t_push": 5, "i": 1}
    ls.close()


# ---------------------------------------------------------------------------------------------
# checkpoint / resume and the out-of-memory path (failures are made on the host)
# ---------------------------------------------------------------------------------------------
@pytest.mark.parametrize("wdt", [gen.F32, gen.BF16])
def test_checkpoint_resume_is_bit_identical(tmp_path, wdt):
    from paper_2506_04531_b200.inputs.gen_cuda import DeviceGenerator
    lay = layouts.decoder_layout("tiny", 2, 64, 300)
    worker_lps = [0, 0, 1, 1]
    hp = dict(K=4, **PAPER_HP)
    events = tr.generate_trace(tr.TraceSpec(P=lay.P, worker_lps=worker_lps, speeds=[1.0, 2.5, 3.0, 1.7],
                                            t_profiled_ms=1.0, n_arrivals=90, K=4))
    cut = 41
    assert any(int(e["kind"]) == tr.PULL for e in events[cut:]) and any(int(e["kind"]) == tr.GPS_RECV for e in events[:cut])
    dg = DeviceGenerator(lay, 17)
    scratch = torch.empty(lay.P, dtype=torch.float32 if wdt == gen.F32 else torch.int16, device="cuda")

    def run(h, evs):
        def producer(index, worker, rnd):
            return dg.worker_result(h.peek(hb.BUF_THETA0, worker), worker, rnd, out=scratch, worker_dtype=wdt)
        return h.replay(evs, producer)

    ref = hb.Halos(dg.theta_init(), worker_lps, lay.numel, worker_dtype=wdt, **hp)
    log_ref = run(ref, events)
    a = hb.Halos(dg.theta_init(), worker_lps, lay.numel, worker_dtype=wdt, **hp)
    run(a, events[:cut])
    path = tmp_path / "state.ckpt"
    a.export_file(path)
    counters = [a.counters(l) for l in (0, 1)]
    a.close()
    b = hb.Halos(torch.zeros(lay.P, device="cuda"), worker_lps, lay.numel, worker_dtype=wdt, **hp)
    b.import_file(path)
    assert [b.counters(l) for l in (0, 1)] == counters
    log_b = run(b, events[cut:])
    for which in range(8):
        n = len(worker_lps) if which == hb.BUF_THETA0 else (1 if which < 2 else 2)
        for idx in range(n):
            assert np.array_equal(ref.read(which, idx).view(np.uint8), b.read(which, idx).view(np.uint8)), (which, idx)
    for f in ("t", "t_last", "gps_iter", "worker_staleness", "gps_lag", "pushed"):
        assert np.array_equal(log_ref[f][cut:], log_b[f])
    # a file of another shape is refused and leaves the state alone
    other = hb.Halos(torch.zeros(64, device="cuda"), [0])
    with pytest.raises(hb.HalosError) as e:
        other.import_file(path)
    assert e.value.status == hb.ERR_INVALID_ARG
    # ... and so is a context with the same shape but other hyperparameters (a different run)
    for change in (dict(K=5), dict(eta_l=0.25), dict(beta_g=0.4), dict(alpha=0.5)):
        odd = hb.Halos(torch.ones(lay.P, device="cuda"), worker_lps, lay.numel, worker_dtype=wdt, **dict(hp, **change))
        with pytest.raises(hb.HalosError) as e:
            odd.import_file(path)
        assert e.value.status == hb.ERR_INVALID_ARG and "hyperparameters" in str(e.value)
        assert odd.counters(0)["t"] == 0 and float(odd.read(hb.BUF_THETA_L, 0, 0, 8).min()) == 1.0   # untouched
        odd.close()
    # pending results cannot be checkpointed
    b.worker_delta(0, scratch)
    with pytest.raises(hb.HalosError) as e:
        b.export_file(tmp_path / "x.ckpt")
    assert e.value.status == hb.ERR_BAD_STATE
    for h in (ref, b, other):
        h.close()


def test_out_of_memory_is_reported_and_cleaned_up():
    P = 1 << 16
    init = torch.zeros(P, device="cuda")
    need = P * 4 * (2 + 5 * 2 + 3)
    for budget in (1024, P * 4 * 3, need - 1):
        with pytest.raises(hb.HalosError) as e:
            hb.Halos(init, [0, 1, 1], alloc_limit_bytes=budget)
        assert e.value.status == hb.ERR_OOM
    h = hb.Halos(init, [0, 1, 1], alloc_limit_bytes=need + (1 << 20))
    assert h.counters(1)["t"] == 0
    # the staging buffer for host-resident results does not fit in the budget: reported, state unchanged
    host = torch.zeros(P).pin_memory()
    h2 = hb.Halos(init, [0], alloc_limit_bytes=P * 4 * 8 + 65536)
    with pytest.raises(hb.HalosError) as e:
        h2.worker_delta_host(0, host)
    assert e.value.status == hb.ERR_OOM and h2.worker_info(0)["pending"] is False
    h.close()
    h2.close()


# ---------------------------------------------------------------------------------------------
# multi-event fusion: batched replay leaves exactly the state and the log of the unbatched replay
# ---------------------------------------------------------------------------------------------
@pytest.mark.parametrize("wdt", [gen.F32, gen.BF16])
@pytest.mark.parametrize("mode", ["flat", "ptrs"])
@pytest.mark.parametrize("max_batch", [2, 3, 4, 6, 8, 99])
def test_batched_replay_is_bit_identical(wdt, mode, max_batch):
    from paper_2506_04531_b200.inputs.gen_cuda import DeviceGenerator
    lay = layouts.ragged_layout("r", [4099, 33, 20001, 5, 8192, 8191, 3])
    worker_lps = [0, 0, 0, 0, 0, 0, 0, 0, 1, 1, 1, 2]
    hp = dict(K=11, **PAPER_HP)
    speeds = [1.0, 1.05, 1.1, 1.15, 1.2, 1.25, 1.3, 3.9, 1.1, 1.2, 3.3, 2.0]
    events = tr.generate_trace(tr.TraceSpec(P=lay.P, worker_lps=worker_lps, speeds=speeds, t_profiled_ms=1.0,
                                            n_arrivals=300, K=11))
    dg = DeviceGenerator(lay, 23)
    tdt = torch.float32 if wdt == gen.F32 else torch.int16
    off = lay.offsets.astype(np.int64)

    def make(h):
        # one result buffer per worker: with batching a result must survive until that worker's next call
        bufs = [torch.empty(lay.P, dtype=tdt, device="cuda") for _ in worker_lps]

        def producer(index, worker, rnd):
            r = dg.worker_result(h.peek(hb.BUF_THETA0, worker), worker, rnd, out=bufs[worker], worker_dtype=wdt)
            if mode == "flat":
                return r
            return [r[off[k]:off[k + 1]] for k in range(lay.n_tensors)]
        return producer

    ref = hb.Halos(dg.theta_init(), worker_lps, lay.numel, worker_dtype=wdt, chunk_elems=1024, **hp)
    log_ref = ref.replay(events, make(ref))
    bat = hb.Halos(dg.theta_init(), worker_lps, lay.numel, worker_dtype=wdt, chunk_elems=1024, **hp)
    bat.timing_enable(True)
    log_bat = bat.replay(events, make(bat), max_batch=max_batch)
    timing = bat.timing_read()
    assert timing["arrive_multi"][0] > 10                      # batches did form
    assert bat.info()["launches"] < ref.info()["launches"]
    for which in range(8):
        n = len(worker_lps) if which == hb.BUF_THETA0 else (1 if which < 2 else 3)
        for idx in range(n):
            assert np.array_equal(ref.read(which, idx).view(np.uint8), bat.read(which, idx).view(np.uint8)), (which, idx)
    for f in ("index", "kind", "lps", "worker", "t", "t_last", "gps_iter", "worker_staleness", "gps_lag", "pushed"):
        assert np.array_equal(log_ref[f], log_bat[f]), f
    for l in range(3):
        assert ref.counters(l) == bat.counters(l)
    ref.close()
    bat.close()


def test_batched_replay_against_oracle_160m_window():
    """Full-size buffers, batched driver, oracle on probe windows (first 300 events of the 160m trace)."""
    from paper_2506_04531_b200.inputs.gen_cuda import DeviceGenerator
    wl = workloads.workload("160m")
    lay = wl.layout
    probes = default_probes(lay, width=4096, n_random=6, seed=9)
    events = wl.trace()[:300]
    ls = Lockstep(lay, wl.worker_lps, wl.hyper(), wl.worker_dtype, wl.seed, probes=probes)
    bufs = [torch.empty(lay.P, dtype=torch.float32, device="cuda") for _ in range(wl.n_workers)]

    def producer(index, worker, rnd):
        return ls.dgen.worker_result(ls.h.peek(hb.BUF_THETA0, worker), worker, rnd, out=bufs[worker])

    ls.h.replay(events, producer, max_batch=4)
    # the oracle side of the lock-step harness, event by event
    for ev in events:
        kind, l, w = int(ev["kind"]), int(ev["lps"]), int(ev["worker"])
        if kind == tr.ARRIVE:
            ls.o.arrive(w, ls._oracle_result(w, ls.o.worker_info(w)["round"]))
        elif kind == tr.GPS_RECV:
            ls.o.gps_recv(l)
        else:
            ls.o.pull(l)
    ls.compare(ls.all_buffers(), FULL_TRACE_TOL)
    assert ls.bit_identical
    ls.close()


# ---------------------------------------------------------------------------------------------
# optional delayed-Nesterov optimizer (the paper's experimental setting: d_l = 16, d_g = 2)
# ---------------------------------------------------------------------------------------------
DN_HP = dict(eta_l=3.2, beta_l=0.9, eta_g=0.3, beta_g=0.5, alpha=0.25, optimizer=hb.OPT_DELAYED_NESTEROV,
             delay_l=16, delay_g=2)


@pytest.mark.parametrize("wdt", [gen.F32, gen.BF16])
@pytest.mark.parametrize("mode", ["flat", "ptrs_misaligned"])
def test_delayed_nesterov_small_shapes(wdt, mode):
    lay = layouts.ragged_layout("r", [4099, 33, 20001, 5, 8192, 8191, 1])
    worker_lps = [0, 0, 1, 1, 1]
    hp = dict(DN_HP, K=5, delay_l=3)
    events = tr.random_trace(worker_lps, 120, 5, seed=77)
    ls = Lockstep(lay, worker_lps, hp, wdt, seed=6, chunk_elems=1024, input_mode=mode)
    ls.run(events, check_every=1, full_check_every=30)
    assert ls.bit_identical and ls.max_err == 0.0
    assert ls.h.counters(0)["i"] >= 4
    ls.close()


def test_delayed_nesterov_toy_config_paper_settings():
    wl = workloads.workload("toy_k4")
    hp = dict(DN_HP, K=wl.K)
    ls = Lockstep(wl.layout, wl.worker_lps, hp, wl.worker_dtype, wl.seed)
    ls.run(wl.trace(), check_every=1, full_check_every=100)
    assert ls.bit_identical and ls.max_err <= PER_EVENT_TOL
    ls.close()


def test_delayed_nesterov_replay_and_checkpoint(tmp_path):
    from paper_2506_04531_b200.inputs.gen_cuda import DeviceGenerator
    lay = layouts.decoder_layout("tiny", 2, 64, 300)
    worker_lps = [0, 0, 1, 1]
    hp = dict(DN_HP, K=4, delay_l=3)
    events = tr.generate_trace(tr.TraceSpec(P=lay.P, worker_lps=worker_lps, speeds=[1.0, 2.5, 3.0, 1.7],
                                            t_profiled_ms=1.0, n_arrivals=90, K=4))
    dg = DeviceGenerator(lay, 19)
    bufs = [torch.empty(lay.P, dtype=torch.float32, device="cuda") for _ in worker_lps]

    def run(h, evs, mb):
        def producer(index, worker, rnd):
            return dg.worker_result(h.peek(hb.BUF_THETA0, worker), worker, rnd, out=bufs[worker])
        return h.replay(evs, producer, max_batch=mb)

    ref = hb.Halos(dg.theta_init(), worker_lps, lay.numel, **hp)
    run(ref, events, 1)
    a = hb.Halos(dg.theta_init(), worker_lps, lay.numel, **hp)
    run(a, events[:37], 4)                 # batched (fused delayed-Nesterov launches) up to the checkpoint
    assert a.batch_info()["multi_launches"] > 0
    a.export_file(tmp_path / "dn.ckpt")
    a.close()
    b = hb.Halos(torch.zeros(lay.P, device="cuda"), worker_lps, lay.numel, **hp)
    b.import_file(tmp_path / "dn.ckpt")
    run(b, events[37:], 1)
    for which in (hb.BUF_THETA_G, hb.BUF_M_G, hb.BUF_ACC_G):
        assert np.array_equal(ref.read(which).view(np.uint32), b.read(which).view(np.uint32))
    for l in (0, 1):
        for which in (hb.BUF_THETA_L, hb.BUF_M_L, hb.BUF_ACC_L, hb.BUF_ANCHOR):
            assert np.array_equal(ref.read(which, l).view(np.uint32), b.read(which, l).view(np.uint32))
    other_delay = hb.Halos(torch.zeros(lay.P, device="cuda"), worker_lps, lay.numel, **dict(hp, delay_l=4))
    with pytest.raises(hb.HalosError) as e:
        other_delay.import_file(tmp_path / "dn.ckpt")  # another refresh schedule: refused
    assert e.value.status == hb.ERR_INVALID_ARG
    other_delay.close()
    plain = hb.Halos(torch.zeros(lay.P, device="cuda"), worker_lps, lay.numel, K=4)
    with pytest.raises(hb.HalosError):
        plain.import_file(tmp_path / "dn.ckpt")       # other optimizer: refused
    with pytest.raises(hb.HalosError):
        plain.read(hb.BUF_ACC_G)
    for h in (ref, b, plain):
        h.close()


def test_guard_zones_detect_an_out_of_bounds_write():
    P = 1001                                   # odd size: the tail guard starts right after the last element
    h = hb.Halos(torch.zeros(P, device="cuda"), [0], flags=hb.FLAG_GUARD)
    assert h.check_guards() == -1
    th = h.peek(hb.BUF_THETA_L, 0)
    # simulate a stray write one element past the end of theta (3rd state buffer: Theta, m_g, theta_0)
    end_addr = th.data_ptr() + 4 * P
    iface = {"shape": (1,), "typestr": "<f4", "data": (end_addr, False), "version": 2}
    holder = type("_Mem", (), {"__cuda_array_interface__": iface})()
    torch.as_tensor(holder, device="cuda").fill_(1.0)
    assert h.check_guards() == 2
    h.close()
    plain = hb.Halos(torch.zeros(8, device="cuda"), [0])
    with pytest.raises(hb.HalosError):
        plain.check_guards()
    plain.close()


# ---------------------------------------------------------------------------------------------
# materialised deltas: the borrow of theta_H ends when halos_worker_delta has been enqueued
# ---------------------------------------------------------------------------------------------
@pytest.mark.parametrize("wdt", [gen.F32, gen.BF16])
@pytest.mark.parametrize("mode", ["flat", "ptrs_misaligned"])
def test_materialised_delta_matches_oracle(wdt, mode):
    lay = layouts.ragged_layout("r", [4099, 33, 20001, 5, 8192, 8191, 1])
    worker_lps = [0, 0, 1, 1, 1]
    events = tr.random_trace(worker_lps, 90, 4, seed=55)
    ls = Lockstep(lay, worker_lps, dict(K=4, **PAPER_HP), wdt, seed=12, chunk_elems=1024, input_mode=mode,
                  flags=hb.FLAG_MATERIALISE_DELTA | hb.FLAG_GUARD)
    ls.run(events, check_every=1, full_check_every=30)
    assert ls.bit_identical and ls.max_err == 0.0 and ls.h.check_guards() == -1
    ls.close()


def test_materialised_delta_frees_the_callers_buffer():
    from oracle import HalosOracle
    lay = layouts.flat_layout("x", 100_003)
    init = gen.theta_init(lay, 9)
    h = hb.Halos(torch.from_numpy(init).cuda(), [0, 0, 0], K=3, flags=hb.FLAG_MATERIALISE_DELTA, **PAPER_HP)
    o = HalosOracle(init, [0, 0, 0], K=3, **PAPER_HP)
    scratch = torch.empty(lay.P, device="cuda")
    pinned = torch.empty(lay.P).pin_memory()
    for rnd in range(3):
        results = [gen.worker_result(o.buffer("th0", w), lay, 9, w, rnd) for w in range(3)]
        # all three results pass through ONE device buffer (and one pinned host buffer): each is overwritten
        # by the next before any of them has been applied
        scratch.copy_(torch.from_numpy(results[0]))
        h.worker_delta(0, scratch)
        scratch.copy_(torch.from_numpy(results[1]))
        h.worker_delta(1, scratch)
        pinned.copy_(torch.from_numpy(results[2]))
        h.worker_delta_host(2, pinned)
        torch.cuda.synchronize()
        pinned.zero_()
        scratch.zero_()
        for w in (1, 2, 0):
            due = h.lps_apply(0, w)
            assert due == o.arrive(w, results[w])
            if due:
                h.lps_push(0)
                h.gps_merge(0)
                o.gps_recv(0)
                h.lps_pull(0)
                o.pull(0)
    for which, name in ((hb.BUF_THETA_L, "th"), (hb.BUF_M_L, "ml"), (hb.BUF_ANCHOR, "anchor")):
        assert np.array_equal(h.read(which, 0).view(np.uint32), o.buffer(name, 0).view(np.uint32))
    assert np.array_equal(h.read(hb.BUF_THETA_G).view(np.uint32), o.buffer("Theta").view(np.uint32))
    h.close()


# ---------------------------------------------------------------------------------------------
# random call sequences, legal and illegal, against a reference state machine and the oracle
# ---------------------------------------------------------------------------------------------
@pytest.mark.parametrize("seed", range(3))
def test_api_fuzz_statuses_and_state(seed):
    from oracle import HalosOracle
    rng = np.random.default_rng(500 + seed)
    lay = layouts.ragged_layout("f", [129, 7, 64, 1, 300])
    worker_lps = [0, 0, 1, 2, 2]
    n_lps, K = 3, 10 ** 6                       # pushes happen when the fuzzer says so, not on a window
    init = gen.theta_init(lay, 70 + seed)
    h = hb.Halos(torch.from_numpy(init).cuda(), worker_lps, lay.numel, K=K, flags=hb.FLAG_GUARD, **PAPER_HP)
    o = HalosOracle(init, worker_lps, K=K, **PAPER_HP)
    pending = {}                                # worker -> result (numpy) registered but not applied
    keep = {}
    phase = [hb.IDLE] * n_lps
    fetched = []
    n_ok = n_bad = 0
    for step in range(700):
        op = int(rng.integers(0, 7))
        l, w = int(rng.integers(0, n_lps + 1)), int(rng.integers(0, len(worker_lps) + 1))   # sometimes out of range
        if rng.random() < 0.85:                 # mostly well-formed arguments, so that the state really advances
            l, w = min(l, n_lps - 1), min(w, 4)
            if op == 1 and rng.random() < 0.8:
                l = worker_lps[w]
        want, call = hb.OK, None
        if op == 0:
            res = gen.worker_result(o.buffer("th0", min(w, 4)), lay, 70 + seed, min(w, 4), step)
            cand = torch.from_numpy(res).cuda()
            call = lambda: h.worker_delta(w, cand)
            want = hb.ERR_INVALID_ARG if w >= 5 else (hb.ERR_BAD_STATE if w in pending else hb.OK)
            if want == hb.OK:
                pending[w] = res
                keep[w] = cand                  # borrowed by the library until the apply: keep it alive
        elif op == 1:
            call = lambda: h.lps_apply(l, w)
            if l >= n_lps or w >= 5 or worker_lps[w] != l:
                want = hb.ERR_INVALID_ARG
            elif w not in pending:
                want = hb.ERR_BAD_STATE
            else:
                o.arrive(w, pending.pop(w))
        elif op == 2:
            call = lambda: h.lps_push(l)
            want = hb.ERR_INVALID_ARG if l >= n_lps else (hb.ERR_BAD_STATE if phase[l] != hb.IDLE else hb.OK)
            if want == hb.OK:
                o.push(l)
                phase[l] = hb.PUSHED
        elif op == 3:
            call = lambda: h.gps_merge(l)
            want = hb.ERR_INVALID_ARG if l >= n_lps else (hb.ERR_BAD_STATE if phase[l] != hb.PUSHED else hb.OK)
            if want == hb.OK:
                o.gps_recv(l)
                phase[l] = hb.ANSWERED
        elif op == 4:
            call = lambda: h.lps_pull(l)
            want = hb.ERR_INVALID_ARG if l >= n_lps else (hb.ERR_BAD_STATE if phase[l] != hb.ANSWERED else hb.OK)
            if want == hb.OK:
                o.pull(l)
                phase[l] = hb.IDLE
        elif op == 5:                           # GPS update and merge as one launch
            call = lambda: h.gps_merge_pull(l)
            want = hb.ERR_INVALID_ARG if l >= n_lps else (hb.ERR_BAD_STATE if phase[l] != hb.PUSHED else hb.OK)
            if want == hb.OK:
                o.gps_recv(l)
                o.pull(l)
                phase[l] = hb.IDLE
        else:                                   # the worker's start model copied out while later updates run on
            dst = torch.empty(lay.P, dtype=torch.float32).pin_memory()
            call = lambda: h.worker_fetch_host(w, dst)
            want = hb.ERR_INVALID_ARG if w >= 5 else hb.OK
            if want == hb.OK:
                fetched.append((dst, o.buffer("th0", w).copy()))
        if want == hb.OK:
            call()
            n_ok += 1
        else:
            with pytest.raises(hb.HalosError) as e:
                call()
            assert e.value.status == want, (step, op, l, w)
            n_bad += 1
    assert n_ok > 150 and n_bad > 150
    h.fetch_sync()
    assert len(fetched) > 20
    for dst, want_th0 in fetched:
        assert np.array_equal(dst.numpy().view(np.uint32), want_th0.view(np.uint32))
    for l in range(n_lps):
        assert h.counters(l) == o.counters(l)
        for which, name in ((hb.BUF_THETA_L, "th"), (hb.BUF_M_L, "ml"), (hb.BUF_ANCHOR, "anchor"),
                            (hb.BUF_OUTBOX, "outbox"), (hb.BUF_INBOX, "inbox")):
            assert np.array_equal(h.read(which, l).view(np.uint32), o.buffer(name, l).view(np.uint32)), (name, l)
    assert np.array_equal(h.read(hb.BUF_THETA_G).view(np.uint32), o.buffer("Theta").view(np.uint32))
    assert np.array_equal(h.read(hb.BUF_M_G).view(np.uint32), o.buffer("Mg").view(np.uint32))
    for w in range(5):
        assert np.array_equal(h.read(hb.BUF_THETA0, w).view(np.uint32), o.buffer("th0", w).view(np.uint32))
    assert h.check_guards() == -1
    h.close()


# ---------------------------------------------------------------------------------------------
# plumbing variants: a non-default stream, the library's own cudaMalloc, two contexts interleaved
# ---------------------------------------------------------------------------------------------
def test_side_stream_own_allocator_and_interleaved_contexts():
    from oracle import HalosOracle
    lay = layouts.ragged_layout("p", [5000, 3, 12345, 64])
    init = gen.theta_init(lay, 41)
    worker_lps = [0, 1, 1]
    side = torch.cuda.Stream()
    init_dev = torch.from_numpy(init).cuda()
    torch.cuda.synchronize()
    with torch.cuda.stream(side):
        a = hb.Halos(init_dev, worker_lps, lay.numel, K=2, stream=side, **PAPER_HP)
    b = hb.Halos(init_dev, worker_lps, lay.numel, K=2, use_torch_allocator=False, **PAPER_HP)
    oa = HalosOracle(init, worker_lps, K=2, **PAPER_HP)
    events = tr.random_trace(worker_lps, 60, 2, seed=3)
    keep = []
    for ev in events:
        kind, l, w = int(ev["kind"]), int(ev["lps"]), int(ev["worker"])
        if kind == tr.ARRIVE:
            res = gen.worker_result(oa.buffer("th0", w), lay, 41, w, oa.worker_info(w)["round"])
            t = torch.from_numpy(res).cuda()
            torch.cuda.synchronize()               # the input is complete before either stream reads it
            keep.append(t)
            for h in (a, b):                       # the two contexts take turns, each on its own stream
                h.worker_delta(w, t)
                if h.lps_apply(l, w):
                    h.lps_push(l)
            oa.arrive(w, res)
        elif kind == tr.GPS_RECV:
            a.gps_merge(l); b.gps_merge(l); oa.gps_recv(l)
        else:
            a.lps_pull(l); b.lps_pull(l); oa.pull(l)
    for h in (a, b):
        for l in (0, 1):
            assert np.array_equal(h.read(hb.BUF_THETA_L, l).view(np.uint32), oa.buffer("th", l).view(np.uint32))
        assert np.array_equal(h.read(hb.BUF_THETA_G).view(np.uint32), oa.buffer("Theta").view(np.uint32))
        h.close()


def test_streaming_replay_keeps_batches_across_calls():
    from paper_2506_04531_b200.inputs.gen_cuda import DeviceGenerator
    lay = layouts.ragged_layout("r", [4099, 33, 20001, 5, 8192, 8191, 3])
    worker_lps = [0, 0, 0, 0, 0, 0, 1, 1, 1, 2]
    hp = dict(K=9, **PAPER_HP)
    speeds = [1.0, 1.05, 1.1, 1.15, 1.2, 3.9, 1.1, 1.2, 3.3, 2.0]
    events = tr.generate_trace(tr.TraceSpec(P=lay.P, worker_lps=worker_lps, speeds=speeds, t_profiled_ms=1.0,
                                            n_arrivals=240, K=9))
    dg = DeviceGenerator(lay, 29)

    def make(h):
        bufs = [torch.empty(lay.P, dtype=torch.float32, device="cuda") for _ in worker_lps]
        return lambda index, worker, rnd: dg.worker_result(h.peek(hb.BUF_THETA0, worker), worker, rnd, out=bufs[worker])

    ref = hb.Halos(dg.theta_init(), worker_lps, lay.numel, chunk_elems=1024, **hp)
    log_ref = ref.replay(events, make(ref))
    one = hb.Halos(dg.theta_init(), worker_lps, lay.numel, chunk_elems=1024, **hp)
    one.replay(events, make(one), max_batch=8)
    st = hb.Halos(dg.theta_init(), worker_lps, lay.numel, chunk_elems=1024, **hp)
    prod = make(st)
    logs = []
    for a in range(0, len(events), 5):                       # five events per call: far shorter than a batch window
        logs.append(st.replay(events[a:a + 5], prod, max_batch=8, keep_queued=True))
    queued_before = st.info()["launches"]
    st.flush()
    cut = hb.Halos(dg.theta_init(), worker_lps, lay.numel, chunk_elems=1024, **hp)
    prod_cut = make(cut)
    for a in range(0, len(events), 5):
        cut.replay(events[a:a + 5], prod_cut, max_batch=8)   # same calls, but every call flushes
    # streaming fuses as well as one big call (except where a call boundary separates a GPS_RECV from the PULL
    # that directly follows it: those run as two launches instead of one) and much better than calls that flush
    kinds, lpss = events["kind"], events["lps"]
    split_pairs = sum(1 for k in range(4, len(events) - 1, 5)
                      if kinds[k] == tr.GPS_RECV and kinds[k + 1] == tr.PULL and lpss[k] == lpss[k + 1])
    assert st.info()["launches"] <= one.info()["launches"] + 1 + split_pairs
    assert st.info()["launches"] < 0.9 * cut.info()["launches"]
    log_st = np.concatenate(logs)
    for f in ("kind", "lps", "worker", "t", "t_last", "gps_iter", "worker_staleness", "gps_lag", "pushed"):
        assert np.array_equal(log_ref[f], log_st[f]), f
    for h in (one, st, cut):
        for which in range(8):
            n = len(worker_lps) if which == hb.BUF_THETA0 else (1 if which < 2 else 3)
            for idx in range(n):
                assert np.array_equal(ref.read(which, idx).view(np.uint8), h.read(which, idx).view(np.uint8)), (which, idx)
    # any entry point that looks at the state launches what is queued
    st2 = hb.Halos(dg.theta_init(), worker_lps, lay.numel, chunk_elems=1024, **hp)
    st2.replay(events[:3], make(st2), max_batch=8, keep_queued=True)
    ref2 = hb.Halos(dg.theta_init(), worker_lps, lay.numel, chunk_elems=1024, **hp)
    ref2.replay(events[:3], make(ref2))
    l0 = int(events[0]["lps"])
    assert np.array_equal(st2.read(hb.BUF_THETA_L, l0).view(np.uint32), ref2.read(hb.BUF_THETA_L, l0).view(np.uint32))
    for h in (ref, one, st, cut, st2, ref2):
        h.close()


def test_replay_stops_at_the_first_bad_event_and_keeps_what_came_before():
    P = 4096
    init = torch.linspace(-1, 1, P, device="cuda")
    good = hb.Halos(init, [0, 0, 1], K=3, **PAPER_HP)
    bad = hb.Halos(init, [0, 0, 1], K=3, **PAPER_HP)
    res = [init + 0.01 * (w + 1) for w in range(3)]
    ev = np.zeros(6, dtype=tr.EVENT_DTYPE)
    ev["kind"] = [tr.ARRIVE, tr.ARRIVE, tr.ARRIVE, tr.PULL, tr.ARRIVE, tr.ARRIVE]
    ev["lps"] = [0, 1, 0, 1, 0, 0]
    ev["worker"] = [0, 2, 1, 0, 0, 1]
    good.replay(ev[:3], lambda i, w, r: res[w], max_batch=4)
    with pytest.raises(hb.HalosError) as e:                  # event 3: PULL for an LPS that never pushed
        bad.replay(ev, lambda i, w, r: res[w], max_batch=4)
    assert e.value.status == hb.ERR_BAD_STATE and "event 3" in str(e.value)
    for l in (0, 1):
        assert bad.counters(l) == good.counters(l)
        assert np.array_equal(bad.read(hb.BUF_THETA_L, l), good.read(hb.BUF_THETA_L, l))
    # a failing producer aborts the replay and its exception reaches the caller
    def broken(i, w, r):
        raise KeyError("no result for this worker")
    with pytest.raises(KeyError):
        bad.replay(ev[4:5], broken)
    assert bad.counters(0) == good.counters(0) and not bad.worker_info(0)["pending"]
    ev2 = ev[:1].copy()
    ev2["lps"] = 9
    with pytest.raises(hb.HalosError) as e:
        bad.replay(ev2, lambda i, w, r: res[w])
    assert e.value.status == hb.ERR_INVALID_ARG
    # an arrival that names a worker of another LPS is refused BEFORE the producer is asked: nothing is
    # registered, so no borrowed pointer outlives the failed call
    ev3 = ev[:1].copy()
    ev3["lps"], ev3["worker"] = 1, 0
    asked = []
    with pytest.raises(hb.HalosError) as e:
        bad.replay(ev3, lambda i, w, r: asked.append(w) or res[w])
    assert e.value.status == hb.ERR_INVALID_ARG and not asked
    assert not bad.worker_info(0)["pending"]
    # the same for an arrival that would close a window while the previous round trip is still in flight
    # (the equality test of Alg. 1 line 13 never lets that happen by itself: it takes a push made by hand)
    late = hb.Halos(init, [0, 0, 1], K=2, **PAPER_HP)
    late.replay(ev[:1], lambda i, w, r: res[w])              # t = 1
    late.lps_push(0)                                         # round trip in flight, t_last still 0
    with pytest.raises(hb.HalosError) as e:                  # t = 2 would close the window of K = 2
        late.replay(ev[2:3], lambda i, w, r: asked.append(w) or res[w])
    assert e.value.status == hb.ERR_BAD_STATE and not asked and not late.worker_info(1)["pending"]
    late.close()
    good.close()
    bad.close()


@pytest.mark.parametrize("wdt", [gen.F32, gen.BF16])
@pytest.mark.parametrize("delay_l", [1, 3, 16])
def test_batched_replay_with_delayed_nesterov(wdt, delay_l):
    """Fused launches under the delayed-Nesterov optimizer: refreshes may fall anywhere inside a batch."""
    from paper_2506_04531_b200.inputs.gen_cuda import DeviceGenerator
    lay = layouts.ragged_layout("r", [4099, 33, 20001, 5, 8192, 8191, 3])
    worker_lps = [0, 0, 0, 0, 0, 0, 0, 0, 1, 1, 1, 2]
    hp = dict(DN_HP, K=11, delay_l=delay_l)
    speeds = [1.0, 1.05, 1.1, 1.15, 1.2, 1.25, 1.3, 3.9, 1.1, 1.2, 3.3, 2.0]
    events = tr.generate_trace(tr.TraceSpec(P=lay.P, worker_lps=worker_lps, speeds=speeds, t_profiled_ms=1.0,
                                            n_arrivals=300, K=11))
    dg = DeviceGenerator(lay, 31)
    tdt = torch.float32 if wdt == gen.F32 else torch.int16

    def make(h):
        bufs = [torch.empty(lay.P, dtype=tdt, device="cuda") for _ in worker_lps]
        return lambda index, worker, rnd: dg.worker_result(h.peek(hb.BUF_THETA0, worker), worker, rnd, out=bufs[worker],
                                                           worker_dtype=wdt)
    ref = hb.Halos(dg.theta_init(), worker_lps, lay.numel, worker_dtype=wdt, chunk_elems=1024, **hp)
    log_ref = ref.replay(events, make(ref))
    bat = hb.Halos(dg.theta_init(), worker_lps, lay.numel, worker_dtype=wdt, chunk_elems=1024, **hp)
    log_bat = bat.replay(events, make(bat), max_batch=8)
    assert bat.batch_info()["multi_launches"] > 10
    for which in list(range(8)) + [hb.BUF_ACC_L, hb.BUF_ACC_G]:
        n = len(worker_lps) if which == hb.BUF_THETA0 else (1 if which in (0, 1, hb.BUF_ACC_G) else 3)
        for idx in range(n):
            assert np.array_equal(ref.read(which, idx).view(np.uint8), bat.read(which, idx).view(np.uint8)), (which, idx)
    for f in ("t", "t_last", "gps_iter", "worker_staleness", "gps_lag", "pushed"):
        assert np.array_equal(log_ref[f], log_bat[f]), f
    ref.close()
    bat.close()
