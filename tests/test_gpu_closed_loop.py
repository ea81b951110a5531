"""Closing the loop: workers that really run H local SGD steps (Alg. 1 lines 22-24) on a synthetic
quadratic objective drive the hierarchy through the CUDA library.  Checks that the GPS model
converges to the optimum of the average objective, that the oracle agrees bit for bit when its own
workers run the same steps, and the qualitative roles of alpha the paper describes."""
from __future__ import annotations

import numpy as np
import pytest
import torch

from oracle import HalosOracle
from paper_2506_04531_b200 import binding as hb
from paper_2506_04531_b200.inputs import gen, layouts, trace as tr

pytestmark = pytest.mark.gpu

H_STEPS, ETA_W = 8, 0.05


def _targets(P, n_workers, seed):
    """Worker i minimises F_i = 1/2 |theta - c_i|^2; the c_i scatter around a common optimum c."""
    lay = layouts.flat_layout("q", P)
    c = gen.unit_noise(gen.stream_key(seed, 50, 0), 0, P)
    offs = [gen.unit_noise(gen.stream_key(seed, 60 + w, 0), 0, P) * np.float32(0.2) for w in range(n_workers)]
    mean_off = np.mean(offs, axis=0).astype(np.float32)
    cs = [(c + o - mean_off).astype(np.float32) for o in offs]      # average of the c_i is c (to rounding)
    return lay, c, cs


def _local_sgd_np(s0, c):
    x = s0.copy()
    for _ in range(H_STEPS):
        x = x - np.float32(ETA_W) * (x - c)          # three separately rounded fp32 operations per step
    return x


def _local_sgd_torch(s0, c):
    x = s0.clone()
    for _ in range(H_STEPS):
        g = x - c
        g = g * ETA_W
        x = x - g
    return x


def _run(alpha, K, n_arrivals=400, with_oracle=False, P=4096, seed=3):
    worker_lps = [0, 0, 0, 1, 1, 1, 2, 2]
    lay, c, cs = _targets(P, len(worker_lps), seed)
    hp = dict(eta_l=0.2, beta_l=0.9, eta_g=0.15, beta_g=0.5, alpha=alpha, K=K)
    events = tr.generate_trace(tr.TraceSpec(P=P, worker_lps=worker_lps, speeds=[4, 1.3, 2.2, 3.1, 1.0, 2.9, 3.7, 1.8],
                                            t_profiled_ms=1.0, n_arrivals=n_arrivals, K=K))
    init = np.zeros(P, np.float32)
    h = hb.Halos(torch.from_numpy(init).cuda(), worker_lps, **hp)
    o = HalosOracle(init, worker_lps, dtype=np.float32, **hp) if with_oracle else None
    cs_dev = [torch.from_numpy(x).cuda() for x in cs]
    dist = []
    for ev in events:
        kind, l, w = int(ev["kind"]), int(ev["lps"]), int(ev["worker"])
        if kind == tr.ARRIVE:
            res = _local_sgd_torch(h.peek(hb.BUF_THETA0, w), cs_dev[w])
            h.worker_delta(w, res)
            if h.lps_apply(l, w):
                h.lps_push(l)
            if o is not None:
                o.arrive(w, _local_sgd_np(o.buffer("th0", w), cs[w]))
        elif kind == tr.GPS_RECV:
            h.gps_merge(l)
            if o is not None:
                o.gps_recv(l)
            dist.append(float(np.linalg.norm(h.read(hb.BUF_THETA_G) - c)))
        else:
            h.lps_pull(l)
            if o is not None:
                o.pull(l)
    out = dict(dist=dist, c=c, Theta=h.read(hb.BUF_THETA_G), th=[h.read(hb.BUF_THETA_L, l) for l in range(3)],
               oracle=o, norm_c=float(np.linalg.norm(c)))
    h.close()
    return out


def test_hierarchy_converges_on_quadratic_and_matches_oracle():
    r = _run(alpha=0.25, K=4, with_oracle=True)
    d = r["dist"]
    assert len(d) >= 30
    assert d[0] > 0.5 * r["norm_c"]                   # starts far away (Theta_0 = 0)
    assert d[-1] < 0.05 * r["norm_c"]                 # ends at the optimum of the average objective
    o = r["oracle"]
    assert np.array_equal(r["Theta"].view(np.uint32), o.buffer("Theta").view(np.uint32))
    for l in range(3):
        assert np.array_equal(r["th"][l].view(np.uint32), o.buffer("th", l).view(np.uint32))


def test_merging_weight_roles():
    # alpha = 0: the LPSs never see the global model; each converges to ITS region's optimum and the
    # regions stay apart.  alpha > 0 pulls them together.
    spread = {}
    for alpha in (0.0, 0.25, 1.0):
        r = _run(alpha=alpha, K=4)
        th = r["th"]
        spread[alpha] = float(np.mean([np.linalg.norm(th[a] - th[b]) for a, b in ((0, 1), (0, 2), (1, 2))]))
    assert spread[0.25] < 0.5 * spread[0.0]
    assert spread[1.0] < spread[0.0]
