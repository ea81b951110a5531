"""Pins for the optional delayed-Nesterov optimizer of the oracle.

The paper uses this optimizer in its experiments but does not define it (it cites the
Async-Local-SGD work); the reading is therefore unpinned by the paper itself.  What is pinned:
  * the one property the paper states (hyperparameter table, Appendix D): the rule "effectively
    divides the learning rate by the delay interval" -- under a constant pseudo-gradient the mean
    step per update is eps g / (d (1 - beta));
  * delay 1 is textbook Nesterov SGD (checked against torch.optim.SGD(nesterov=True));
  * an independent scalar interpreter of the same reading, on random hierarchical traces;
  * structural facts: momentum only moves on refresh updates, the accumulator holds the sum since
    the last refresh and is cleared by it.
"""
from __future__ import annotations

import numpy as np
import pytest
import torch

import oracle
from oracle import HalosOracle
from paper_2506_04531_b200.inputs import trace as tr

DN = oracle.OPT_DELAYED_NESTEROV


def _feed(o, w, disp):
    """Arrive with a result that displaces the worker's snapshot by (the fp32-rounded) disp; returns what was fed."""
    s0 = o.buffer("th0", w).astype(np.float64)
    thH = (s0 + disp).astype(np.float32)
    pushed = o.arrive(w, thH)
    return thH.astype(np.float64) - s0, pushed


def test_delay_one_is_textbook_nesterov_sgd():
    rng = np.random.default_rng(0)
    P, eps, beta = 16, 0.3, 0.8
    init = rng.normal(size=P).astype(np.float32)
    o = HalosOracle(init, [0], eta_l=eps, beta_l=beta, K=10 ** 6, dtype=np.float64, optimizer=DN, delay_l=1)
    x = torch.tensor(init.astype(np.float64), requires_grad=True)
    opt = torch.optim.SGD([x], lr=eps, momentum=beta, nesterov=True)
    for _ in range(40):
        fed, _ = _feed(o, 0, rng.normal(size=P) * 0.05)
        x.grad = torch.tensor(-fed)               # pseudo-gradient = minus the displacement
        opt.step()
        np.testing.assert_allclose(o.buffer("th", 0), x.detach().numpy(), rtol=1e-12, atol=1e-14)


@pytest.mark.parametrize("delay,eps,beta", [(2, 0.3, 0.5), (16, 3.2, 0.9), (4, 1.0, 0.0)])
def test_mean_step_is_learning_rate_over_delay(delay, eps, beta):
    # constant displacement delta: after the momentum has settled, every block of `delay` updates moves
    # the model by eps delta / (1 - beta), i.e. a mean step of (eps / delay) delta / (1 - beta)
    P = 4
    delta = np.array([2.0 ** -12, -3 * 2.0 ** -13, 5 * 2.0 ** -14, 2.0 ** -11])
    o = HalosOracle(np.zeros(P, np.float32), [0], eta_l=eps, beta_l=beta, K=10 ** 6, dtype=np.float64,
                    optimizer=DN, delay_l=delay)
    blocks, fed_hist, marks = 160, [], []      # beta^160 < 1e-7: the momentum has settled
    for n in range(1, blocks * delay + 1):
        fed, _ = _feed(o, 0, delta)
        fed_hist.append(fed)
        if n % delay == 0:
            marks.append(o.buffer("th", 0).copy())
    per_block = marks[-1] - marks[-2]
    mean_fed = np.mean(fed_hist[-delay:], axis=0)
    np.testing.assert_allclose(per_block / delay, (eps / delay) * mean_fed / (1 - beta), rtol=2e-4)
    # and the intended constant is what was fed up to the fp32 snapshot rounding
    np.testing.assert_allclose(mean_fed, delta, rtol=1e-3)


def test_momentum_moves_only_on_refresh_and_accumulator_resets():
    rng = np.random.default_rng(1)
    P, d = 8, 4
    o = HalosOracle(np.zeros(P, np.float32), [0], eta_l=0.4, beta_l=0.7, K=10 ** 6, dtype=np.float64,
                    optimizer=DN, delay_l=d)
    acc = np.zeros(P)
    for n in range(1, 21):
        m_before, th_before = o.buffer("ml", 0).copy(), o.buffer("th", 0).copy()
        fed, _ = _feed(o, 0, rng.normal(size=P) * 0.01)
        acc += fed
        if n % d:
            np.testing.assert_array_equal(o.buffer("ml", 0), m_before)
            np.testing.assert_allclose(o.buffer("acc", 0), acc, rtol=1e-15, atol=1e-18)
            np.testing.assert_allclose(o.buffer("th", 0) - th_before, (0.4 / d) * fed, rtol=1e-12, atol=1e-16)
        else:
            np.testing.assert_allclose(o.buffer("ml", 0), 0.7 * m_before + acc / d, rtol=1e-14, atol=1e-18)
            assert np.all(o.buffer("acc", 0) == 0)
            acc[:] = 0


class _Interp:
    """Independent scalar interpreter of the hierarchy with delayed Nesterov servers (gradient form)."""

    def __init__(self, init, worker_lps, eps_l, beta_l, d_l, eps_g, beta_g, d_g, alpha, K):
        n_lps = max(worker_lps) + 1
        self.wl, self.K, self.alpha = worker_lps, K, alpha
        self.l = [dict(x=list(init), m=[0.0] * len(init), acc=[0.0] * len(init), n=0, t_last=0, anchor=list(init),
                       out=None, inn=None) for _ in range(n_lps)]
        self.g = dict(x=list(init), m=[0.0] * len(init), acc=[0.0] * len(init), n=0)
        self.start = [list(init) for _ in worker_lps]
        self.hp_l, self.hp_g = (eps_l, beta_l, d_l), (eps_g, beta_g, d_g)

    @staticmethod
    def _opt(srv, disp, eps, beta, d):
        srv["n"] += 1
        for j, dj in enumerate(disp):
            g = -dj
            srv["acc"][j] += g
            if srv["n"] % d:
                srv["x"][j] -= (eps / d) * g
            else:
                srv["m"][j] = beta * srv["m"][j] + srv["acc"][j] / d
                srv["x"][j] -= eps * (beta * srv["m"][j] + g / d)
                srv["acc"][j] = 0.0

    def arrive(self, w, disp):
        s = self.l[self.wl[w]]
        self._opt(s, disp, *self.hp_l)
        self.start[w] = list(s["x"])
        if s["n"] - s["t_last"] == self.K:
            s["out"] = [a - b for a, b in zip(s["x"], s["anchor"])]
            return True
        return False

    def gps(self, l):
        s = self.l[l]
        self._opt(self.g, s["out"], *self.hp_g)
        s["out"], s["inn"] = None, list(self.g["x"])

    def pull(self, l):
        s = self.l[l]
        s["t_last"] = s["n"]
        s["x"] = [(1 - self.alpha) * a + self.alpha * b for a, b in zip(s["x"], s["inn"])]
        s["anchor"], s["inn"] = list(s["x"]), None


@pytest.mark.parametrize("seed", range(4))
def test_random_traces_against_independent_interpreter(seed):
    rng = np.random.default_rng(40 + seed)
    P = 5
    worker_lps = [[0, 0, 1], [0, 1, 1, 2], [0, 0], [0, 1, 2, 2, 1, 0]][seed]
    K, d_l, d_g = [4, 3, 2, 5][seed], [2, 3, 16, 4][seed], [2, 1, 3, 2][seed]
    hp = dict(eta_l=float(rng.uniform(0.1, 3)), beta_l=float(rng.uniform(0, 0.95)), eta_g=float(rng.uniform(0.05, 1)),
              beta_g=float(rng.uniform(0, 0.9)), alpha=float(rng.uniform(0, 1)))
    init = rng.normal(size=P).astype(np.float32)
    o = HalosOracle(init, worker_lps, K=K, dtype=np.float64, optimizer=DN, delay_l=d_l, delay_g=d_g, **hp)
    it = _Interp([float(v) for v in init], worker_lps, hp["eta_l"], hp["beta_l"], d_l, hp["eta_g"], hp["beta_g"], d_g,
                 hp["alpha"], K)
    for ev in tr.random_trace(worker_lps, 150, K, seed):
        kind, l, w = int(ev["kind"]), int(ev["lps"]), int(ev["worker"])
        if kind == tr.ARRIVE:
            fed, pushed = _feed(o, w, rng.normal(size=P) * 0.02)
            assert it.arrive(w, list(fed)) == pushed
        elif kind == tr.GPS_RECV:
            o.gps_recv(l)
            it.gps(l)
        else:
            o.pull(l)
            it.pull(l)
        for ll in range(max(worker_lps) + 1):
            np.testing.assert_allclose(o.buffer("th", ll), it.l[ll]["x"], rtol=1e-10, atol=1e-13)
        np.testing.assert_allclose(o.buffer("Theta"), it.g["x"], rtol=1e-10, atol=1e-13)
        np.testing.assert_allclose(o.buffer("Mg"), [-v for v in it.g["m"]], rtol=1e-10, atol=1e-13)


def test_paper_rule_unchanged_by_the_new_fields():
    # OPT_PAPER ignores delays entirely
    rng = np.random.default_rng(2)
    init = rng.normal(size=8).astype(np.float32)
    a = HalosOracle(init, [0], K=3, dtype=np.float32)
    b = HalosOracle(init, [0], K=3, dtype=np.float32, delay_l=5, delay_g=7)
    for _ in range(7):
        r = (a.buffer("th0", 0) + rng.normal(size=8).astype(np.float32) * np.float32(0.01)).astype(np.float32)
        pa, pb = a.arrive(0, r), b.arrive(0, r)
        assert pa == pb
        if pa:
            for o in (a, b):
                o.gps_recv(0)
                o.pull(0)
    np.testing.assert_array_equal(a.buffer("th", 0), b.buffer("th", 0))
    np.testing.assert_array_equal(a.buffer("Theta"), b.buffer("Theta"))
