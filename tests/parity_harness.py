"""Drives the CUDA library (through its C ABI binding) and the CPU oracle in lock-step on the same
seeded trace and the same seeded inputs, and compares their state.

The oracle replays an index subset ("probes": a list of [lo, hi) ranges of the packed parameter
vector, or everything); this is legitimate because every step of the method is elementwise.  Its
inputs come from the numpy generator applied to ITS OWN worker snapshots, the GPU's inputs from
the CUDA twin applied to the GPU's snapshots: no value ever flows from the CUDA path to the oracle.
"""
from __future__ import annotations

from typing import List, Optional, Sequence, Tuple

import numpy as np
import torch

import oracle as oracle_mod
from oracle import HalosOracle
from paper_2506_04531_b200 import binding as hb
from paper_2506_04531_b200.inputs import gen, trace as tr
from paper_2506_04531_b200.inputs.gen_c import HostGenerator
from paper_2506_04531_b200.inputs.gen_cuda import DeviceGenerator
from paper_2506_04531_b200.inputs.layouts import Layout

PER_EVENT_TOL = 1e-6   # max relative error per event (stated tolerance of the benchmark spec)
FULL_TRACE_TOL = 1e-5  # after the full trace

_BUF = {"Theta": hb.BUF_THETA_G, "Mg": hb.BUF_M_G, "th": hb.BUF_THETA_L, "ml": hb.BUF_M_L,
        "anchor": hb.BUF_ANCHOR, "outbox": hb.BUF_OUTBOX, "inbox": hb.BUF_INBOX, "th0": hb.BUF_THETA0,
        "acc": hb.BUF_ACC_L, "acc_g": hb.BUF_ACC_G}


def rel_error(got: np.ndarray, want: np.ndarray) -> float:
    """max_j |g_j - o_j| / max(|o_j|, 1e-3 rms(o)); inf if anything is not finite."""
    g, o = got.astype(np.float64), want.astype(np.float64)
    if not (np.isfinite(g).all() and np.isfinite(o).all()):
        return float("inf")
    if g.size == 0:
        return 0.0
    floor = 1e-3 * float(np.sqrt(np.mean(o * o)))
    den = np.maximum(np.abs(o), max(floor, 1e-30))
    return float(np.max(np.abs(g - o) / den))


def default_probes(layout: Layout, width: int = 8192, n_random: int = 16, random_width: int = 65536, edge: int = 65536,
                   seed: int = 0) -> List[Tuple[int, int]]:
    """The first and last `edge` elements, `width` elements centred on EVERY tensor boundary, and `n_random`
    random windows of `random_width` elements; overlapping windows are merged."""
    P = layout.P
    off = layout.offsets.astype(np.int64)
    spans = [(0, min(P, edge)), (max(0, P - edge), P)]
    for b in off[1:-1]:
        spans.append((max(0, int(b) - width // 2), min(P, int(b) + width // 2)))
    rng = np.random.default_rng(seed)
    for s in rng.integers(0, max(1, P - random_width), size=n_random):
        spans.append((int(s), min(P, int(s) + random_width)))
    spans.sort()
    merged = []
    for lo, hi in spans:
        if merged and lo <= merged[-1][1]:
            merged[-1] = (merged[-1][0], max(hi, merged[-1][1]))
        else:
            merged.append((lo, hi))
    return merged


class Lockstep:
    def __init__(self, layout: Layout, worker_lps: Sequence[int], hyper: dict, worker_dtype: int, seed: int,
                 probes: Optional[List[Tuple[int, int]]] = None, chunk_elems: int = 0, flags: int = 0,
                 input_mode: str = "flat", device: str = "cuda", sigma_table=None):
        self.layout, self.seed, self.worker_dtype = layout, seed, worker_dtype
        self.worker_lps = list(worker_lps)
        self.input_mode = input_mode
        self.sigma_table = sigma_table
        P = layout.P
        self.probes = probes if probes is not None else [(0, P)]
        self.full = probes is None
        self.dgen = DeviceGenerator(layout, seed, device=device, sigma_table=sigma_table)
        self.hgen = HostGenerator(layout, seed, sigma_table=sigma_table)   # C twin of gen.py (cross-checked bit for bit)
        init_dev = self.dgen.theta_init()
        self.h = hb.Halos(init_dev, worker_lps, layout.numel, worker_dtype=worker_dtype, flags=flags,
                          chunk_elems=chunk_elems, **hyper)
        del init_dev
        init_cpu = np.concatenate([self.hgen.theta_init(lo, hi) for lo, hi in self.probes])
        self.o = HalosOracle(init_cpu, worker_lps, worker_dtype=worker_dtype, dtype=np.float32, **hyper)
        if not self.full:
            idx = np.concatenate([np.arange(lo, hi, dtype=np.int64) for lo, hi in self.probes])
            self.idx_dev = torch.from_numpy(idx).to(device)
        wdt = torch.float32 if worker_dtype == gen.F32 else torch.int16
        self._wdt = wdt
        if input_mode == "flat":
            self.thH = torch.empty(P, dtype=wdt, device=device)
        else:
            # one separately allocated tensor per layout tensor; "ptrs_misaligned" shifts every
            # second tensor by one element so that its address is not 16-byte aligned
            self.thH_parts = []
            for k, n in enumerate(layout.numel):
                pad = 1 if (input_mode == "ptrs_misaligned" and k % 2 == 1) else 0
                buf = torch.empty(int(n) + pad + 8, dtype=wdt, device=device)
                self.thH_parts.append(buf[pad:pad + int(n)])
        self.delayed = hyper.get("optimizer", 0) == hb.OPT_DELAYED_NESTEROV
        self.inbox_iter = [0] * (max(worker_lps) + 1)
        self.log = []
        self.bit_identical = True
        self.max_err = 0.0

    # ------------------------------------------------------------------ inputs
    def _gpu_result(self, w: int, rnd: int):
        s0 = self.h.peek(hb.BUF_THETA0, w)
        if self.input_mode == "flat":
            self.dgen.worker_result(s0, w, rnd, out=self.thH, worker_dtype=self.worker_dtype)
            return self.thH, None
        off = self.layout.offsets.astype(np.int64)
        for k, part in enumerate(self.thH_parts):
            if part.numel():
                self.dgen.worker_result(s0[off[k]:off[k + 1]], w, rnd, out=part, worker_dtype=self.worker_dtype,
                                        lo=int(off[k]))
        return None, self.thH_parts

    def _oracle_result(self, w: int, rnd: int) -> np.ndarray:
        s0 = self.o.buffer("th0", w)
        parts, pos = [], 0
        for lo, hi in self.probes:
            parts.append(self.hgen.worker_result(s0[pos:pos + hi - lo], w, rnd, lo, self.worker_dtype))
            pos += hi - lo
        return np.concatenate(parts)

    # ------------------------------------------------------------------ events
    def step(self, ev, use_fused_replay: bool = False) -> dict:
        kind, l, w = int(ev["kind"]), int(ev["lps"]), int(ev["worker"])
        rec = {"kind": kind, "lps": l, "worker": w, "pushed": False}
        if kind == tr.ARRIVE:
            rnd_g = self.h.worker_info(w)["round"]
            rnd_o = self.o.worker_info(w)["round"]
            assert rnd_g == rnd_o
            rec["worker_staleness"] = self.o.counters(l)["t"] - self.o.worker_info(w)["sched_t"]
            assert rec["worker_staleness"] == self.h.counters(l)["t"] - self.h.worker_info(w)["sched_t"]
            flat, parts = self._gpu_result(w, rnd_g)
            self.h.worker_delta(w, flat, parts)
            due = self.h.lps_apply(l, w)
            if due:
                self.h.lps_push(l)
            pushed = self.o.arrive(w, self._oracle_result(w, rnd_o))
            assert due == pushed
            rec["pushed"] = pushed
        elif kind == tr.GPS_RECV:
            self.h.gps_merge(l)
            self.o.gps_recv(l)
            self.inbox_iter[l] = self.o.counters(l)["i"]
        else:
            rec["gps_lag"] = self.o.counters(l)["i"] - self.inbox_iter[l]
            self.h.lps_pull(l)
            self.o.pull(l)
        cg, co = self.h.counters(l), self.o.counters(l)
        assert cg == co, (cg, co)
        rec.update(t=co["t"], t_last=co["t_last"], gps_iter=co["i"])
        self.log.append(rec)
        return rec

    def written_by(self, rec) -> List[Tuple[str, int]]:
        kind, l, w = rec["kind"], rec["lps"], rec["worker"]
        if kind == tr.ARRIVE:
            out = [("th", l), ("ml", l), ("th0", w)] + ([("acc", l)] if self.delayed else [])
            if rec["pushed"]:
                out.append(("outbox", l))
            return out
        if kind == tr.GPS_RECV:
            return [("Theta", 0), ("Mg", 0), ("inbox", l)] + ([("acc_g", 0)] if self.delayed else [])
        return [("th", l), ("anchor", l)]

    def all_buffers(self) -> List[Tuple[str, int]]:
        n_lps = max(self.worker_lps) + 1
        out = [("Theta", 0), ("Mg", 0)]
        for l in range(n_lps):
            out += [(b, l) for b in ("th", "ml", "anchor", "outbox", "inbox")]
        out += [("th0", w) for w in range(len(self.worker_lps))]
        if self.delayed:
            out += [("acc_g", 0)] + [("acc", l) for l in range(n_lps)]
        return out

    # ------------------------------------------------------------------ comparison
    def gpu_values(self, name: str, idx: int) -> np.ndarray:
        t = self.h.peek(_BUF[name], idx)
        if not self.full:
            t = t.index_select(0, self.idx_dev)
        a = t.cpu().numpy()
        if name == "th0" and self.worker_dtype == gen.BF16:
            return a.view(np.uint16)
        return a

    def compare(self, buffers, tol: float) -> float:
        worst = 0.0
        for name, idx in buffers:
            g = self.gpu_values(name, idx)
            o = self.o.buffer(name, idx)
            if name == "th0" and self.worker_dtype == gen.BF16:
                same = np.array_equal(g, o)
                err = 0.0 if same else rel_error(gen.bf16_bits_to_f32(g), gen.bf16_bits_to_f32(o))
            else:
                same = np.array_equal(g.view(np.uint32), o.view(np.uint32))
                err = 0.0 if same else rel_error(g, o)
            self.bit_identical &= bool(same)
            worst = max(worst, err)
            assert err <= tol, f"{name}[{idx}]: relative error {err:.3e} > {tol:.1e}"
        self.max_err = max(self.max_err, worst)
        return worst

    def run(self, events, check_every: int = 1, full_check_every: int = 0):
        for n, ev in enumerate(events):
            rec = self.step(ev)
            if check_every and (n % check_every == 0):
                self.compare(self.written_by(rec), PER_EVENT_TOL)
            if full_check_every and (n + 1) % full_check_every == 0:
                self.compare(self.all_buffers(), FULL_TRACE_TOL)
        self.compare(self.all_buffers(), FULL_TRACE_TOL)
        return self

    def close(self):
        self.h.close()
        self.o.close()
