"""The synthetic workloads: a parameter layout, a cluster shape and an arrival trace each.

They stand in for the paper's simulated geo-distributed cluster (four regions, heterogeneous
worker speeds, profiled step times of Pythia-70M/160M/410M on one H100: 238.4, 623.0 and
1589.7 ms) -- only the structure that reaches the server-side update path is kept.
"""
from __future__ import annotations

import json
from dataclasses import dataclass
from pathlib import Path
from typing import List, Optional, Sequence

import numpy as np

from . import gen
from .layouts import Layout, named_layout
from .trace import GBPS_TO_GPS_REGION, PAPER_WORKER_SPEEDS, TraceSpec, generate_trace, worker_speeds


@dataclass
class Workload:
    name: str
    layout: Layout
    n_workers: int
    n_lps: int
    worker_dtype: int
    t_profiled_ms: float
    n_arrivals: int
    seed: int
    K: int = 32
    eta_l: float = 0.2
    beta_l: float = 0.9
    eta_g: float = 0.15
    beta_g: float = 0.5
    alpha: float = 0.25
    slow_region_factor: float = 1.0   # speeds of the last region's workers are divided by this
    fixed_speeds: Optional[Sequence[float]] = None   # e.g. the paper's 16 worker speeds
    fixed_worker_lps: Optional[Sequence[int]] = None  # non-uniform grouping of workers under LPSs
    lps_gbps: Optional[Sequence[float]] = None        # LPS -> GPS link of each LPS (default: by region l % 4)
    dyn_updates: bool = False
    bandwidth_scale: float = 1.0
    optimizer: int = 0                # 0: the update rule the paper defines; 1: delayed Nesterov (its experiments)
    delay_l: int = 1
    delay_g: int = 1

    @property
    def worker_lps(self) -> List[int]:
        if self.fixed_worker_lps is not None:
            return list(self.fixed_worker_lps)
        per = self.n_workers // self.n_lps
        return [w // per for w in range(self.n_workers)]

    @property
    def speeds(self) -> List[float]:
        if self.fixed_speeds is not None:
            return list(self.fixed_speeds)
        s = worker_speeds(self.n_workers, self.seed)
        if self.slow_region_factor != 1.0:
            wl = self.worker_lps
            s = [v / self.slow_region_factor if wl[w] == self.n_lps - 1 else v for w, v in enumerate(s)]
        return s

    def trace(self, n_arrivals: int | None = None) -> np.ndarray:
        return generate_trace(TraceSpec(
            P=self.layout.P, worker_lps=self.worker_lps, speeds=self.speeds,
            t_profiled_ms=self.t_profiled_ms, n_arrivals=n_arrivals or self.n_arrivals, K=self.K,
            lps_gbps=self.lps_gbps, dyn_updates=self.dyn_updates, bandwidth_scale=self.bandwidth_scale))

    def hyper(self) -> dict:
        hp = dict(eta_l=self.eta_l, beta_l=self.beta_l, eta_g=self.eta_g, beta_g=self.beta_g,
                  alpha=self.alpha, K=self.K)
        if self.optimizer:
            hp.update(optimizer=self.optimizer, delay_l=self.delay_l, delay_g=self.delay_g)
        return hp


CONFIG_DIR = Path(__file__).resolve().parent / "configs"
_INT_KEYS = {"n_workers", "n_lps", "n_arrivals", "seed", "K", "delay_l", "delay_g"}
_FLOAT_KEYS = {"t_profiled_ms", "eta_l", "beta_l", "eta_g", "beta_g", "alpha", "slow_region_factor", "bandwidth_scale"}
_REQUIRED = ("name", "layout", "n_workers", "n_lps", "worker_dtype", "t_profiled_ms", "n_arrivals", "seed")


def parse_config(text: str) -> dict:
    """`key = value` lines ('#' starts a comment) or a JSON object -> dict of raw values."""
    text = text.strip()
    if text.startswith("{"):
        return dict(json.loads(text))
    out = {}
    for n, line in enumerate(text.splitlines(), 1):
        line = line.split("#", 1)[0].strip()
        if not line:
            continue
        if "=" not in line:
            raise ValueError(f"line {n}: expected key = value")
        k, v = (x.strip() for x in line.split("=", 1))
        if k in out:
            raise ValueError(f"line {n}: {k} given twice")
        out[k] = v
    return out


def from_config(cfg: dict) -> Workload:
    """Builds a workload from a parsed configuration.  Keys: name, layout (toy | 70m | 160m | 410m | 1p4b, or
    'decoder' with layers/d/vocab, or 'flat' with P), n_workers, n_lps, worker_dtype (f32 | bf16), t_profiled_ms,
    n_arrivals, seed; optional K, eta_l, beta_l, eta_g, beta_g, alpha (default: the paper's selected values),
    slow_region_factor, bandwidth_scale, dyn_updates, optimizer (paper | delayed_nesterov), delay_l, delay_g."""
    cfg = dict(cfg)
    missing = [k for k in _REQUIRED if k not in cfg]
    if missing:
        raise ValueError(f"configuration lacks {missing}")
    lay = str(cfg.pop("layout"))
    if lay == "decoder":
        from .layouts import decoder_layout
        layout = decoder_layout(str(cfg["name"]), int(cfg.pop("layers")), int(cfg.pop("d")), int(cfg.pop("vocab")))
    elif lay == "flat":
        from .layouts import flat_layout
        layout = flat_layout(str(cfg["name"]), int(cfg.pop("P")))
    else:
        layout = named_layout(lay)
    wd = str(cfg.pop("worker_dtype")).lower()
    if wd not in ("f32", "bf16"):
        raise ValueError("worker_dtype must be f32 or bf16")
    kw = {}
    for k, v in cfg.items():
        if k == "name":
            continue
        if k in _INT_KEYS:
            kw[k] = int(v)
        elif k in _FLOAT_KEYS:
            kw[k] = float(v)
        elif k == "dyn_updates":
            kw[k] = str(v).lower() in ("1", "true", "yes")
        elif k == "optimizer":
            kw[k] = {"paper": 0, "delayed_nesterov": 1}[str(v)]
        else:
            raise ValueError(f"unknown configuration key {k!r}")
    n_workers, n_lps = kw.pop("n_workers"), kw.pop("n_lps")
    if n_workers % n_lps:
        raise ValueError("n_workers must be a multiple of n_lps")
    return Workload(str(cfg["name"]), layout, n_workers, n_lps, gen.F32 if wd == "f32" else gen.BF16,
                    kw.pop("t_profiled_ms"), kw.pop("n_arrivals"), **kw)


def load(path) -> Workload:
    """A workload from a configuration file (key = value lines or JSON)."""
    return from_config(parse_config(Path(path).read_text()))


def workload(name: str) -> Workload:
    """toy | toy_k4 | 70m | 160m | 160m_dn | 410m | 70m_f32_small | paper_cluster | paper_cluster_small |
    hetero_grouping_small  (hyperparameters: the paper's selected values).  The four benchmark configurations
    toy, 70m, 160m and 410m are read from the files in configs/."""
    if name in ("toy", "70m", "160m", "410m"):
        return load(CONFIG_DIR / f"{name}.cfg")
    if name == "toy_k4":
        return Workload("toy_k4", named_layout("toy"), 4, 2, gen.F32, 10.0, 200, seed=1, K=4)
    if name == "160m_dn":
        # the 160M configuration under the optimizer and the selected values of the paper's experiments:
        # delayed Nesterov with d_l = 16, eta_l = 16 x 0.2, d_g = 2, eta_g = 2 x 0.15
        return Workload("160m_dn", named_layout("160m"), 16, 4, gen.F32, 623.0, 2000, seed=3,
                        eta_l=3.2, eta_g=0.3, optimizer=1, delay_l=16, delay_g=2)
    if name == "paper_cluster":
        # the paper's own simulated cluster: 4 regions x 4 workers with its 16 worker speeds, one LPS
        # per region, dynamic local updates, 160M layout
        return Workload("paper_cluster", named_layout("160m"), 16, 4, gen.F32, 623.0, 2000, seed=7,
                        fixed_speeds=PAPER_WORKER_SPEEDS, dyn_updates=True)
    if name == "paper_cluster_small":
        # same cluster structure on a 2^20-parameter vector (cheap enough to check every event)
        return Workload("paper_cluster_small", named_layout("toy"), 16, 4, gen.F32, 238.4, 400, seed=7, K=8,
                        fixed_speeds=PAPER_WORKER_SPEEDS, dyn_updates=True)
    if name == "hetero_grouping_small":
        # heterogeneous regions with 2, 4, 4, 6 workers under "consistent grouping": 1, 2, 2, 3 LPSs
        # (two workers each), K = 8, twice the link bandwidth
        wl_map = [l for l in range(8) for _ in range(2)]
        region_of_lps = [0, 1, 1, 2, 2, 3, 3, 3]
        return Workload("hetero_grouping_small", named_layout("toy"), 16, 8, gen.F32, 238.4, 400, seed=8, K=8,
                        fixed_speeds=PAPER_WORKER_SPEEDS, fixed_worker_lps=wl_map,
                        lps_gbps=[GBPS_TO_GPS_REGION[r] for r in region_of_lps], bandwidth_scale=2.0)
    if name == "70m_f32_small":
        # small-memory configuration (~4 GB on the device): the 70M layout with fp32 copies, 4 workers on
        # 1 LPS; every buffer is still larger than L2, and K = 8 makes pushes, GPS updates and merges
        # occur within the first few events.  For GPUs with little free memory and for counter captures.
        return Workload("70m_f32_small", named_layout("70m"), 4, 1, gen.F32, 238.4, 200, seed=6, K=8)
    raise KeyError(name)


SWEEP_SIZES = (1 << 20, 1 << 22, 1 << 24, 1 << 26, 70_426_624, 162_322_944, 1 << 28, 405_334_016, 1 << 30)
