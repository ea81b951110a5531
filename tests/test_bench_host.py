"""Host-side logic of the benchmark: trace windows, the oracle timing leg, the reference arm's JSON
line, and the multi-rank reduction (max time, summed units) under a 2-process gloo group."""
from __future__ import annotations

import json
import os
import subprocess
import sys
from pathlib import Path

import numpy as np

ROOT = Path(__file__).resolve().parent.parent
sys.path.insert(0, str(ROOT))


def test_window_events_and_oracle_sample():
    import bench
    from paper_2506_04531_b200.inputs import workloads, trace as tr
    wl = workloads.workload("toy")
    ev = bench.window_events(5, 64, wl)
    assert len(ev) == 320 and np.all(np.diff(ev["time_ns"]) >= 0)
    ev2 = bench.window_events(20, 64, wl)            # longer than the configured 200 arrivals
    assert len(ev2) == 1280 and np.array_equal(ev2[:200], ev[:200])
    rate, desc, spent, done = bench.oracle_sample(wl, ev[:40], 1 << 14, budget_s=5.0)
    assert done == 40 and rate > 1e5 and "index slice" in desc
    all_rate, cores = bench.oracle_sample_all_cores(wl, ev[:40], 1 << 14, budget_s=5.0)
    assert cores >= 1 and all_rate > 1e5


def _rank_main(rank, world, port, out_dir):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    import torch.distributed as dist
    sys.path.insert(0, str(ROOT))
    import bench
    dist.init_process_group("gloo", rank=rank, world_size=world)
    t, u = bench.reduce_over_ranks(dist, 10.0 + 5.0 * rank, 100.0 * (rank + 1))
    Path(out_dir, f"r{rank}.json").write_text(json.dumps([t, u]))
    dist.destroy_process_group()


def test_reduce_over_ranks_gloo(tmp_path):
    import torch.multiprocessing as mp
    port = 29500 + (os.getpid() % 2000)
    mp.spawn(_rank_main, args=(2, port, str(tmp_path)), nprocs=2, join=True)
    for r in range(2):
        t, u = json.loads(Path(tmp_path, f"r{r}.json").read_text())
        assert t == 15.0 and u == 300.0
    import bench
    assert bench.reduce_over_ranks(None, 3.0, 7.0) == (3.0, 7.0)


def test_reference_arm_line():
    out = subprocess.run([sys.executable, str(ROOT / "bench.py"), "--impl", "reference", "--workload", "toy",
                          "--steps", "1", "--warmup", "0", "--events-per-step", "16"],
                         check=True, capture_output=True, text=True, cwd=str(ROOT)).stdout.strip().splitlines()[-1]
    line = json.loads(out)
    assert line["impl"] == "reference" and line["metric"] == "params_updated_per_sec" and line["value"] > 0
    assert line["cpu_baseline"]["kind"] == "oracle" and line["e2e"]["h2d_bytes_per_step"] == 0


def _shard_main(rank, world, port, out_dir):
    """Index-sharded replicas: every rank replays the same trace on its own contiguous slice of the
    parameter vector; no exchange is needed on the data path (the method is elementwise)."""
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    import torch
    import torch.distributed as dist
    sys.path.insert(0, str(ROOT))
    from oracle import HalosOracle
    from paper_2506_04531_b200.inputs import gen, layouts, trace as tr
    dist.init_process_group("gloo", rank=rank, world_size=world)
    lay = layouts.ragged_layout("s", [1000, 37, 4096, 3, 2000])
    P = lay.P
    lo, hi = rank * P // world, (rank + 1) * P // world
    worker_lps = [0, 0, 1, 1]
    events = tr.random_trace(worker_lps, 80, 3, seed=4)
    o = HalosOracle(gen.theta_init(lay, 5, lo, hi), worker_lps, K=3)
    for ev in events:
        kind, l, w = int(ev["kind"]), int(ev["lps"]), int(ev["worker"])
        if kind == tr.ARRIVE:
            o.arrive(w, gen.worker_result(o.buffer("th0", w), lay, 5, w, o.worker_info(w)["round"], lo, hi))
        elif kind == tr.GPS_RECV:
            o.gps_recv(l)
        else:
            o.pull(l)
    mine = torch.from_numpy(np.concatenate([o.buffer("Theta"), o.buffer("th", 1)]).copy())
    assert P % world == 0                      # equal shards, so a plain all_gather collects the result
    parts = [torch.empty_like(mine) for _ in range(world)]
    dist.all_gather(parts, mine)               # only to collect the answer; the replay itself exchanged nothing
    if rank == 0:
        np.save(Path(out_dir, "gathered.npy"), np.concatenate([p.numpy() for p in parts]))
    dist.destroy_process_group()


def test_index_sharded_replicas_gloo(tmp_path):
    import torch.multiprocessing as mp
    from oracle import HalosOracle
    from paper_2506_04531_b200.inputs import gen, layouts, trace as tr
    port = 31500 + (os.getpid() % 2000)
    mp.spawn(_shard_main, args=(2, port, str(tmp_path)), nprocs=2, join=True)
    got = np.load(tmp_path / "gathered.npy")
    lay = layouts.ragged_layout("s", [1000, 37, 4096, 3, 2000])
    P = lay.P
    worker_lps = [0, 0, 1, 1]
    o = HalosOracle(gen.theta_init(lay, 5), worker_lps, K=3)
    for ev in tr.random_trace(worker_lps, 80, 3, seed=4):
        kind, l, w = int(ev["kind"]), int(ev["lps"]), int(ev["worker"])
        if kind == tr.ARRIVE:
            o.arrive(w, gen.worker_result(o.buffer("th0", w), lay, 5, w, o.worker_info(w)["round"]))
        elif kind == tr.GPS_RECV:
            o.gps_recv(l)
        else:
            o.pull(l)
    half = P // 2
    want = np.concatenate([o.buffer("Theta")[:half], o.buffer("th", 1)[:half], o.buffer("Theta")[half:], o.buffer("th", 1)[half:]])
    assert np.array_equal(got.view(np.uint32), want.view(np.uint32))


def test_step_length_is_shared_by_both_arms_and_kernel_table():
    import bench
    from paper_2506_04531_b200 import binding as hb
    from paper_2506_04531_b200.inputs import workloads
    wl = workloads.workload("160m")
    # a function of the arguments only (never of the free memory of whichever machine runs the arm)
    assert bench.events_per_step(wl, 20, 0) == bench.events_per_step(wl, 20, 0) == 11
    assert bench.events_per_step(wl, 10, 0) == 23 and bench.events_per_step(wl, 10, 8) == 8
    assert bench.events_per_step(workloads.workload("toy"), 10, 0) == 128
    rec = np.zeros(4, dtype=hb.LAUNCH_RECORD_DTYPE)
    rec["kind"], rec["events"], rec["bytes_per_param"], rec["ms"] = [0, 0, 5, 6], [1, 1, 3, 2], [28, 36, 52, 36], [1.0, 1.0, 2.0, 1.0]
    t = bench.kernel_table(rec, 10 ** 9, elapsed_ms=10.0)
    assert t["arrive"]["launches"] == 2 and t["arrive"]["bytes_per_param"] == 32.0 and abs(t["arrive"]["GBps"] - 32000.0) < 1e-6
    assert t["arrive_multi"]["events"] == 3 and abs(t["arrive_multi"]["GBps"] - 26000.0) < 1e-6
    assert t["gps_pull"]["share_of_step"] == 0.1 and t["push"]["launches"] == 0 and t["push"]["GBps"] is None
    s = bench.spread([3.0, 1.0, 2.0])
    assert (s["median"], s["min"], s["max"], s["n"]) == (2.0, 1.0, 3.0, 3) and s["rel_spread"] == 1.0
