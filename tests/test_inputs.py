"""Host-side checks of the synthetic input generators: layouts, noise, traces."""
from __future__ import annotations

import numpy as np
import pytest

from paper_2506_04531_b200.inputs import gen, layouts, trace as tr, workloads


def test_layout_sizes():
    want = {"70m": (70_426_624, 76), "160m": (162_322_944, 148), "410m": (405_334_016, 292),
            "1p4b": (1_414_647_808, 292), "toy": (1 << 20, 1)}
    for name, (P, n) in want.items():
        lay = layouts.named_layout(name)
        assert (lay.P, lay.n_tensors) == (P, n)
        assert lay.offsets[-1] == P and len(lay.offsets) == n + 1
    lay = layouts.named_layout("160m")
    d, L, V = 768, 12, 50304
    assert lay.P == 2 * V * d + L * (12 * d * d + 13 * d) + 2 * d
    assert lay.tensors[0].name == "embed_in" and lay.tensors[-1].name == "embed_out"
    assert min(t.numel for t in lay.tensors) == 768


def test_noise_statistics_and_slicing():
    key = gen.stream_key(5, gen.STREAM_WORKER + 3, 17)
    z = gen.unit_noise(key, 0, 1 << 20)
    assert z.dtype == np.float32
    assert abs(float(z.mean())) < 5e-3
    assert abs(float(z.var()) - 1.0) < 5e-3
    assert float(np.abs(z).max()) <= 4.9
    # kurtosis of Irwin-Hall(8) is 3 - 1.2/8 = 2.85
    assert abs(float(((z.astype(np.float64)) ** 4).mean()) - 2.85) < 0.05
    np.testing.assert_array_equal(gen.unit_noise(key, 12345, 23456), z[12345:23456])
    # different streams / rounds / seeds decorrelate
    z2 = gen.unit_noise(gen.stream_key(5, gen.STREAM_WORKER + 3, 18), 0, 1 << 16)
    z3 = gen.unit_noise(gen.stream_key(5, gen.STREAM_WORKER + 4, 17), 0, 1 << 16)
    for other in (z2, z3):
        assert abs(float(np.corrcoef(z[: 1 << 16], other)[0, 1])) < 0.02
    # neighbouring indices decorrelate
    assert abs(float(np.corrcoef(z[:-1], z[1:])[0, 1])) < 5e-3


def test_theta_init_per_tensor_rules():
    lay = layouts.decoder_layout("tiny", 2, 16, 64)
    th = gen.theta_init(lay, 3)
    off = lay.offsets.astype(int)
    for k, t in enumerate(lay.tensors):
        seg = th[off[k]:off[k + 1]]
        if t.kind == layouts.KIND_NORM_WEIGHT:
            assert np.all(seg == 1.0)
        elif t.kind == layouts.KIND_BIAS:
            assert np.all(seg == 0.0)
        else:
            assert 0.015 < float(seg.std()) < 0.025
    np.testing.assert_array_equal(gen.theta_init(lay, 3, 100, 3000), th[100:3000])


def test_worker_result_dtypes_and_scales():
    lay = layouts.decoder_layout("tiny", 1, 32, 128)
    th = gen.theta_init(lay, 1)
    r = gen.worker_result(th, lay, 1, 2, 0)
    d = r.astype(np.float64) - th
    off = lay.offsets.astype(int)
    assert 0.8e-3 < d[off[0]:off[1]].std() < 1.2e-3          # matrix
    assert 0.5e-4 < d[off[1]:off[2]].std() < 1.5e-4          # 1-D tensor
    hb = gen.f32_to_bf16_bits(th)
    rb = gen.worker_result(hb, lay, 1, 2, 0, worker_dtype=gen.BF16)
    assert rb.dtype == np.uint16
    lo, hi = 777, 2222
    np.testing.assert_array_equal(gen.worker_result(hb[lo:hi], lay, 1, 2, 0, lo, hi, gen.BF16), rb[lo:hi])
    # numpy bf16 helpers against the library conversion
    import torch
    x = (np.random.default_rng(0).normal(size=4096) * 0.02).astype(np.float32)
    lib = torch.from_numpy(x).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    np.testing.assert_array_equal(gen.f32_to_bf16_bits(x), lib)
    np.testing.assert_array_equal(gen.bf16_bits_to_f32(lib), torch.from_numpy(x).to(torch.bfloat16).float().numpy())


@pytest.mark.parametrize("name", ["toy", "toy_k4", "70m", "160m", "410m", "paper_cluster", "paper_cluster_small",
                                  "hetero_grouping_small"])
def test_trace_structure(name):
    wl = workloads.workload(name)
    ev = wl.trace()
    kinds = ev["kind"]
    assert int((kinds == tr.ARRIVE).sum()) == wl.n_arrivals
    t = ev["time_ns"]
    assert np.all(np.diff(t) >= 0)
    # replay the counters: pushes fire exactly on windows of K, each LPS alternates G and P
    n_lps = wl.n_lps
    tt, tl, phase = [0] * n_lps, [0] * n_lps, [0] * n_lps
    n_push = 0
    for e in ev:
        k, l = int(e["kind"]), int(e["lps"])
        if k == tr.ARRIVE:
            assert wl.worker_lps[int(e["worker"])] == l
            tt[l] += 1
            if tt[l] - tl[l] == wl.K:
                assert phase[l] == 0
                phase[l] = 1
                n_push += 1
        elif k == tr.GPS_RECV:
            assert phase[l] == 1
            phase[l] = 2
        else:
            assert phase[l] == 2
            phase[l] = 0
            tl[l] = tt[l]
    assert all(p == 0 for p in phase)                     # in-flight round trips were drained
    assert int((kinds == tr.GPS_RECV).sum()) == n_push == int((kinds == tr.PULL).sum())
    if name != "toy":
        assert n_push >= 8
    # regenerating gives the same trace
    np.testing.assert_array_equal(ev, wl.trace())


def test_trace_heterogeneity():
    wl = workloads.workload("410m")
    ev = wl.trace()
    s = wl.speeds
    assert 1.0 / 3.0 <= min(s) and max(s) <= 4.0
    arr = ev[ev["kind"] == tr.ARRIVE]
    per_lps = [int((arr["lps"] == l).sum()) for l in range(4)]
    assert per_lps[3] < min(per_lps[:3])                  # the slowed-down region arrives least often
    # a worker's arrivals are evenly spaced by its round time
    w0 = arr[arr["worker"] == 0]["time_ns"]
    assert len(set(np.diff(w0).tolist())) == 1


def test_paper_cluster_options():
    wl = workloads.workload("paper_cluster_small")
    assert len(wl.speeds) == 16 and max(wl.speeds) == 10.0 and min(wl.speeds) == 1.2
    ev = wl.trace()
    arr = ev[ev["kind"] == tr.ARRIVE]
    # dynamic local updates: every worker needs the same time per round, so arrivals come in
    # synchronous waves of all 16 workers
    counts = [int((arr["worker"] == w).sum()) for w in range(16)]
    assert max(counts) - min(counts) <= 1
    # without them the fastest worker arrives ~8x as often as the slowest (speeds 10.0 vs 1.2)
    spec = tr.TraceSpec(P=wl.layout.P, worker_lps=wl.worker_lps, speeds=wl.speeds, t_profiled_ms=238.4,
                        n_arrivals=400, K=8)
    arr2 = tr.generate_trace(spec)
    arr2 = arr2[arr2["kind"] == tr.ARRIVE]
    c2 = [int((arr2["worker"] == w).sum()) for w in range(16)]
    assert c2[0] > 6 * c2[15]
    # doubling the bandwidth shortens every LPS<->GPS round trip
    g1 = tr.generate_trace(spec)
    spec2 = tr.TraceSpec(P=wl.layout.P, worker_lps=wl.worker_lps, speeds=wl.speeds, t_profiled_ms=238.4,
                         n_arrivals=400, K=8, bandwidth_scale=2.0)
    g2 = tr.generate_trace(spec2)
    rt = lambda g, l: (g[(g["kind"] == tr.PULL) & (g["lps"] == l)]["time_ns"][0]
                       - g[(g["kind"] == tr.GPS_RECV) & (g["lps"] == l)]["time_ns"][0])
    assert rt(g2, 3) * 2 == pytest.approx(rt(g1, 3), rel=1e-6)
    # consistent grouping: 8 LPSs of two workers each, the last three share region 4's slow link
    hg = workloads.workload("hetero_grouping_small")
    assert hg.n_lps == 8 and sorted(set(hg.worker_lps)) == list(range(8))
    assert hg.lps_gbps[5] == hg.lps_gbps[7] == 0.202 and hg.lps_gbps[0] == 100.0


def test_c_generator_equals_numpy_generator():
    from paper_2506_04531_b200.inputs.gen_c import HostGenerator
    for lay in (layouts.decoder_layout("tiny", 2, 64, 300), layouts.ragged_layout("e", [16, 0, 5, 0, 64, 1, 4099])):
        hg = HostGenerator(lay, 77)
        init = gen.theta_init(lay, 77)
        np.testing.assert_array_equal(hg.theta_init().view(np.uint32), init.view(np.uint32))
        lo, hi = 17, lay.P - 9
        np.testing.assert_array_equal(hg.theta_init(lo, hi), init[lo:hi])
        np.testing.assert_array_equal(hg.worker_result(init[lo:hi], 3, 9, lo).view(np.uint32),
                                      gen.worker_result(init[lo:hi], lay, 77, 3, 9, lo, hi).view(np.uint32))
        hb16 = gen.f32_to_bf16_bits(init)
        np.testing.assert_array_equal(hg.worker_result(hb16[lo:hi], 3, 9, lo, gen.BF16),
                                      gen.worker_result(hb16[lo:hi], lay, 77, 3, 9, lo, hi, gen.BF16))


def test_trace_file_round_trip(tmp_path):
    ev = workloads.workload("toy_k4").trace()
    tr.save_trace(tmp_path / "toy.trace", ev)
    assert (tmp_path / "toy.trace").stat().st_size == 16 * len(ev)
    np.testing.assert_array_equal(tr.load_trace(tmp_path / "toy.trace"), ev)
    (tmp_path / "junk").write_bytes(bytes(range(32)))
    with pytest.raises(ValueError):
        tr.load_trace(tmp_path / "junk")


def test_configuration_files_and_reader(tmp_path):
    """The four benchmark configurations are read from key = value files; the reader takes JSON too and
    refuses unknown keys, missing keys and bad values."""
    import json
    import pytest
    from paper_2506_04531_b200.inputs import workloads as W
    want = {"toy": (1 << 20, 4, 2, gen.F32, 200, 1), "70m": (70_426_624, 8, 2, gen.BF16, 1000, 2),
            "160m": (162_322_944, 16, 4, gen.F32, 2000, 3), "410m": (405_334_016, 32, 4, gen.F32, 2000, 4)}
    for name, (P, nw, nl, wd, na, seed) in want.items():
        wl = W.workload(name)
        assert (wl.layout.P, wl.n_workers, wl.n_lps, wl.worker_dtype, wl.n_arrivals, wl.seed) == (P, nw, nl, wd, na, seed)
        assert wl.hyper() == dict(eta_l=0.2, beta_l=0.9, eta_g=0.15, beta_g=0.5, alpha=0.25, K=32)
    assert W.workload("410m").slow_region_factor == 3.0
    cfg = dict(name="x", layout="decoder", layers=2, d=64, vocab=300, n_workers=6, n_lps=3, worker_dtype="bf16",
               t_profiled_ms=5.0, n_arrivals=40, seed=9, K=4, alpha=0.5, optimizer="delayed_nesterov", delay_l=3, delay_g=2)
    (tmp_path / "x.json").write_text(json.dumps(cfg))
    (tmp_path / "x.cfg").write_text("\n".join(f"{k} = {v}  # note" for k, v in cfg.items()))
    a, b = W.load(tmp_path / "x.json"), W.load(tmp_path / "x.cfg")
    assert a == b and a.layout.n_tensors == 28 and a.worker_dtype == gen.BF16 and a.hyper()["delay_l"] == 3
    assert a.worker_lps == [0, 0, 1, 1, 2, 2] and len(a.trace()) >= 40
    for bad in (dict(cfg, colour="red"), {k: v for k, v in cfg.items() if k != "seed"}, dict(cfg, worker_dtype="f16"),
                dict(cfg, n_workers=7)):
        with pytest.raises((ValueError, KeyError)):
            W.from_config(bad)
    with pytest.raises(ValueError):
        W.parse_config("K 4")


def test_metrics_sinks(tmp_path):
    import csv
    import json
    from paper_2506_04531_b200 import binding as hb, metrics
    rec = np.zeros(3, dtype=hb.LAUNCH_RECORD_DTYPE)
    rec["kind"], rec["events"], rec["bytes_per_param"], rec["ms"] = [0, 5, 6], [1, 4, 2], [28, 64, 36], [0.5, 1.0, 0.25]
    assert metrics.write_launch_records(tmp_path / "l.jsonl", rec, 1000) == 3
    rows = [json.loads(x) for x in (tmp_path / "l.jsonl").read_text().splitlines()]
    assert rows[1] == {"launch": 1, "kernel": "arrive_multi", "events": 4, "bytes": 64000, "us": 1000.0, "GBps": 64000 / 1e9 / 1e-3}
    metrics.write_launch_records(tmp_path / "l.csv", rec, 1000)
    got = list(csv.DictReader(open(tmp_path / "l.csv")))
    assert [r["kernel"] for r in got] == ["arrive", "arrive_multi", "gps_pull"]
    log = np.zeros(2, dtype=hb.EVENT_LOG_DTYPE)
    log["kind"], log["t"], log["fused"] = [0, 2], [7, 7], [1, 0]
    metrics.write_event_log(tmp_path / "e.jsonl", log)
    ev = [json.loads(x) for x in (tmp_path / "e.jsonl").read_text().splitlines()]
    assert ev[0]["kind"] == "ARRIVE" and ev[1]["kind"] == "PULL" and ev[0]["t"] == 7 and ev[0]["fused"] == 1
