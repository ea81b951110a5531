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
