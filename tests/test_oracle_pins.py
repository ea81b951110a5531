"""Pins for the CPU oracle: everything here compares it with something other than itself --
exact rational hand expansion, closed forms, reductions to textbook procedures, special cases,
an independently written history-indexed interpreter of Algorithm 1, and library bf16 rounding.
"""
from __future__ import annotations

import struct
from fractions import Fraction as Fr
from pathlib import Path

import numpy as np
import pytest

import oracle
from oracle import HalosOracle
from paper_interpreter import PaperInterpreter
from paper_2506_04531_b200.inputs import trace as tr

GOLDEN = Path(__file__).parent / "golden" / "hand_expansion_p8.txt"


# ----------------------------------------------------------------------------------------------
# R7: exact hand expansion (Alg. 1 lines 1-25 + Appendix E ModelUpdate) on 8 parameters
# ----------------------------------------------------------------------------------------------
def _load_golden():
    rows, bits = [], {}
    for line in GOLDEN.read_text().splitlines():
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        parts = line.split()
        if parts[0] == "bits":
            bits[parts[1]] = [int(x, 16) for x in parts[2:]]
        else:
            rows.append((int(parts[0]), parts[1], [Fr(x) for x in parts[2:]]))
    return rows, bits


_TRACE_R7 = "A0 A2 A1 A0 G0 A2 G1 P0 A1 P1 A0 G0".split()


def _r7_result(w, r, start):
    return [start[j] + Fr((3 * w + 5 * r + 7 * j) % 9 - 4, 16) for j in range(8)]


def _oracle_buf(o, name):
    if name == "Theta":
        return o.buffer("Theta")
    if name == "Mg":
        return o.buffer("Mg")
    return o.buffer(name[:-1], int(name[-1]))


@pytest.mark.parametrize("dtype", [np.float32, np.float64])
def test_hand_expansion_exact(dtype):
    rows, bits = _load_golden()
    by_event = {}
    for ev, name, vals in rows:
        by_event.setdefault(ev, []).append((name, vals))
    Theta0 = [Fr(j - 4, 8) for j in range(8)]
    half = 0.5
    o = HalosOracle(np.array([float(x) for x in Theta0], np.float32), [0, 0, 1], eta_l=half, beta_l=half,
                    eta_g=half, beta_g=half, alpha=0.25, K=2, dtype=dtype)
    it = PaperInterpreter(Theta0, [0, 0, 1], Fr(1, 2), Fr(1, 2), Fr(1, 2), Fr(1, 2), Fr(1, 4), 2, zero=Fr(0))
    rounds = [0, 0, 0]
    expected_push = {3, 6, 11}
    for n, e in enumerate(_TRACE_R7, 1):
        kind, idx = e[0], int(e[1])
        if kind == "A":
            # both sides get the same worker result, built from the exact interpreter's snapshot
            th = _r7_result(idx, rounds[idx], it.start[idx])
            # the oracle's own snapshot must be that same value (fp32 holds it exactly)
            assert [Fr(float(x)) for x in o.buffer("th0", idx)] == it.start[idx]
            rounds[idx] += 1
            p_it = it.arrive(idx, th)
            p_o = o.arrive(idx, np.array([float(x) for x in th], np.float32))
            assert p_it == p_o == (n in expected_push)
        elif kind == "G":
            it.gps_recv(idx)
            o.gps_recv(idx)
        else:
            it.pull(idx)
            o.pull(idx)
        for name, vals in by_event.get(n, []):
            got = [Fr(float(x)) for x in _oracle_buf(o, name)]
            assert got == vals, f"event {n} buffer {name}"
        # interpreter (exact) against the golden rows that it also produces
        for name, vals in by_event.get(n, []):
            if name.startswith("th"):
                assert it.lps_model(int(name[-1])) == vals
            elif name == "Theta":
                assert it.gps_model() == vals
            elif name.startswith("ml"):
                assert [-x for x in it.m_l[int(name[-1])]] == vals
            elif name == "Mg":
                assert [-x for x in it.m_g] == vals
    if dtype == np.float32:
        for name in ("Theta", "th0", "th1"):
            buf = o.buffer("Theta") if name == "Theta" else o.buffer("th", int(name[-1]))
            assert [struct.unpack("<I", struct.pack("<f", float(x)))[0] for x in buf] == bits[name]
    c0, c1 = o.counters(0), o.counters(1)
    assert (c0["t"], c0["t_last"], c0["phase"], c0["i"]) == (5, 3, oracle.ANSWERED, 3)
    assert (c1["t"], c1["t_last"], c1["phase"]) == (2, 2, oracle.IDLE)


# ----------------------------------------------------------------------------------------------
# R4: closed-form geometric momentum sum for a constant displacement (m_0 = 0)
#   theta_T - theta_0 = eta d [ T (1-b+b^2)/(1-b) - b^2 (1-b^T)/(1-b)^2 ],  m_T = d (1-b^T)/(1-b)
# ----------------------------------------------------------------------------------------------
def _closed_form(eta, beta, d, T):
    return eta * d * (T * (1 - beta + beta * beta) / (1 - beta) - beta * beta * (1 - beta ** T) / (1 - beta) ** 2)


@pytest.mark.parametrize("eta,beta", [(0.2, 0.9), (0.15, 0.5), (1.0, 0.0), (0.7, 0.3)])
def test_closed_form_lps_constant_delta(eta, beta):
    # The worker snapshot theta_{t,0} is an fp32 rounding of the model, so the displacement the
    # oracle really sees (fed) differs from the intended constant d by at most half an fp32 ulp
    # of theta (relative 6e-5 of the smallest d here).  Two checks: the constant-d closed form
    # within that perturbation, and the unrolled geometric sum over the fed history at 1e-12:
    #   theta_T = theta_0 + eta sum_t [ (1-b) d_t + sum_{s<=t} b^(t-s+1) d_s ]
    P = 8
    d = np.array([(j + 1) * 2.0 ** -12 for j in range(P)])
    o = HalosOracle(np.zeros(P, np.float32), [0], eta_l=eta, beta_l=beta, K=10 ** 6, dtype=np.float64)
    checkpoints = {1, 2, 10, 32, 200}
    hist = []
    for T in range(1, 201):
        s0 = o.buffer("th0", 0).astype(np.float64)
        thH = (s0 + d).astype(np.float32)
        hist.append(thH.astype(np.float64) - s0)
        o.arrive(0, thH)
        if T in checkpoints:
            th, ml = o.buffer("th", 0), o.buffer("ml", 0)
            ref = np.array([_closed_form(eta, beta, x, T) for x in d])
            np.testing.assert_allclose(th, ref, rtol=2e-4, atol=0)
            np.testing.assert_allclose(ml, d * (1 - beta ** T) / (1 - beta), rtol=2e-4, atol=0)
            total = np.zeros(P)
            for t in range(1, T + 1):
                inner = sum(beta ** (t - s + 1) * hist[s - 1] for s in range(1, t + 1))
                total += (1 - beta) * hist[t - 1] + inner
            np.testing.assert_allclose(th, eta * total, rtol=1e-12, atol=0)
            m_unrolled = sum(beta ** (T - s) * hist[s - 1] for s in range(1, T + 1))
            np.testing.assert_allclose(ml, m_unrolled, rtol=1e-12, atol=0)


def test_closed_form_printed_values():
    # decimal values of the closed form for d = 1e-3 (exact arithmetic), T = 1, 2, 10, 32, 200
    want = {(0.2, 0.9): {1: 2.0e-4, 2: 5.62e-4, 10: 7.6485907296e-3, 32: 4.25962567789e-2, 200: 0.347800000011},
            (0.15, 0.5): {1: 1.5e-4, 2: 3.375e-4, 10: 2.100146484375e-3, 32: 7.05000000003e-3, 200: 4.485e-2}}
    for (eta, beta), tab in want.items():
        for T, v in tab.items():
            assert _closed_form(eta, beta, 1e-3, T) == pytest.approx(v, rel=2e-11)


def test_closed_form_gps_constant_Delta():
    # beta_l = 0, eta_l = 1, K = 1, alpha = 0: the LPS model is T d (dyadic, exact in fp32, so the
    # worker snapshot arithmetic is exact), every round trip pushes exactly Delta = d, and Theta
    # follows the closed form with (eta_g, beta_g) to rounding error.
    P, eta_g, beta_g = 8, 0.15, 0.5
    d = np.array([(j + 1) * 2.0 ** -12 for j in range(P)]) * np.array([1, -1, 1, 1, -1, 1, -1, 1])
    o = HalosOracle(np.zeros(P, np.float32), [0], eta_l=1.0, beta_l=0.0, eta_g=eta_g, beta_g=beta_g,
                    alpha=0.0, K=1, dtype=np.float64)
    for T in range(1, 201):
        s0 = o.buffer("th0", 0).astype(np.float64)
        thH = (s0 + d).astype(np.float32)
        np.testing.assert_array_equal(thH.astype(np.float64) - s0, d)
        assert o.arrive(0, thH) is True
        np.testing.assert_array_equal(o.buffer("outbox", 0), d)
        o.gps_recv(0)
        o.pull(0)
        ref = np.array([_closed_form(eta_g, beta_g, x, T) for x in d])
        np.testing.assert_allclose(o.buffer("Theta"), ref, rtol=1e-12, atol=0)
        np.testing.assert_allclose(o.buffer("Mg"), d * (1 - beta_g ** T) / (1 - beta_g), rtol=1e-12, atol=0)
        np.testing.assert_array_equal(o.buffer("th", 0), T * d)


# ----------------------------------------------------------------------------------------------
# The paper's own identity (Appendix E, first display after the update rules):
#   (1-beta) g + beta m_{t+1} = g + beta^2 m_t
# ----------------------------------------------------------------------------------------------
def test_instantaneous_term_coefficient():
    eta, beta = 0.25, 0.75
    o = HalosOracle(np.zeros(2, np.float32), [0], eta_l=eta, beta_l=beta, K=99, dtype=np.float64)
    d1 = np.array([0.5, -0.25], np.float32)
    o.arrive(0, d1)                       # theta0 = 0, so delta = d1 and m_1 = d1
    th1 = o.buffer("th", 0).copy()
    np.testing.assert_allclose(th1, eta * d1, rtol=1e-15)           # m_0 = 0: step is eta * d
    s0 = o.buffer("th0", 0).astype(np.float64)
    thH = (s0 + np.array([0.125, 0.375])).astype(np.float32)
    d2 = thH.astype(np.float64) - s0
    o.arrive(0, thH)
    th2 = o.buffer("th", 0)
    np.testing.assert_allclose(th2 - th1, eta * (d2 + beta * beta * d1), rtol=1e-14)


# ----------------------------------------------------------------------------------------------
# R1: no momentum, unit rates -> plain (local) SGD on F = 1/2 |theta - c|^2
# ----------------------------------------------------------------------------------------------
def test_reduces_to_local_sgd():
    rng = np.random.default_rng(7)
    P, H, eta_w, n = 16, 8, 0.05, 25
    c = rng.normal(size=P)
    th_init = rng.normal(size=P).astype(np.float32)
    shrink = (1 - eta_w) ** H
    # one LPS, one worker; the hierarchy collapses too with K = 1, beta_g = 0, eta_g = 1, alpha = 1
    o = HalosOracle(th_init, [0], eta_l=1.0, beta_l=0.0, eta_g=1.0, beta_g=0.0, alpha=1.0, K=1, dtype=np.float64)
    for r in range(1, n + 1):
        s0 = o.buffer("th0", 0).astype(np.float64)
        x = s0.copy()
        for _ in range(H):                      # the worker really runs H SGD steps (Alg. 1 lines 22-24)
            x = x - eta_w * (x - c)
        assert o.arrive(0, x.astype(np.float32)) is True
        o.gps_recv(0)
        o.pull(0)
        ref = c + shrink ** r * (th_init.astype(np.float64) - c)
        np.testing.assert_allclose(o.buffer("th", 0), ref, rtol=0, atol=5e-7)
        np.testing.assert_allclose(o.buffer("Theta"), ref, rtol=0, atol=5e-7)
    # after one arrival the LPS model IS the worker's model
    o2 = HalosOracle(th_init, [0], eta_l=1.0, beta_l=0.0, K=100, dtype=np.float64)
    res = (th_init + rng.normal(size=P).astype(np.float32) * np.float32(0.01)).astype(np.float32)
    o2.arrive(0, res)
    np.testing.assert_allclose(o2.buffer("th", 0), res.astype(np.float64), rtol=0, atol=1e-9)


# ----------------------------------------------------------------------------------------------
# R2: N workers from the same start, eta_l = 1/N, no momentum -> the average of their models
# ----------------------------------------------------------------------------------------------
def test_reduces_to_model_averaging():
    rng = np.random.default_rng(11)
    P, N = 32, 4
    th_init = rng.normal(size=P).astype(np.float32)
    results = [(th_init + rng.normal(size=P).astype(np.float32) * np.float32(0.1)).astype(np.float32) for _ in range(N)]
    avg = np.mean([r.astype(np.float64) for r in results], axis=0)
    finals = []
    for order in ([0, 1, 2, 3], [3, 1, 0, 2], [2, 3, 1, 0]):
        o = HalosOracle(th_init, [0] * N, eta_l=1.0 / N, beta_l=0.0, K=100, dtype=np.float64)
        for w in order:
            o.arrive(w, results[w])
        finals.append(o.buffer("th", 0).copy())
        np.testing.assert_allclose(finals[-1], avg, rtol=0, atol=1e-14)
    np.testing.assert_allclose(finals[0], finals[1], rtol=0, atol=1e-15)


# ----------------------------------------------------------------------------------------------
# R3: the pushed Delta holds exactly the K displacements since the last merge
# ----------------------------------------------------------------------------------------------
def test_window_of_K_updates():
    P, K = 8, 3
    rng = np.random.default_rng(5)
    o = HalosOracle(np.zeros(P, np.float32), [0, 0], eta_l=1.0, beta_l=0.0, eta_g=0.5, beta_g=0.5, alpha=0.5,
                    K=K, dtype=np.float64)
    fed = []

    def arrive(w):
        s0 = o.buffer("th0", w).astype(np.float64)
        thH = (s0 + rng.integers(-8, 9, size=P) / 64.0).astype(np.float32)
        fed.append(thH.astype(np.float64) - s0)
        return o.arrive(w, thH)

    assert not arrive(0) and not arrive(1)
    assert arrive(0)                                            # third update closes the window
    np.testing.assert_allclose(o.buffer("outbox", 0), fed[0] + fed[1] + fed[2], atol=1e-15)
    assert not arrive(1) and not arrive(0)                      # in flight: no second push (t - t_last != K)
    o.gps_recv(0)
    assert not arrive(1)
    o.pull(0)
    assert o.counters(0)["t_last"] == 6
    n0 = len(fed)
    assert not arrive(0) and not arrive(1)
    assert arrive(1)
    # updates 4-6 happened while Delta was in flight and are in no Delta
    np.testing.assert_allclose(o.buffer("outbox", 0), fed[n0] + fed[n0 + 1] + fed[n0 + 2], atol=1e-14)
    with pytest.raises(oracle.OracleError):
        o.pull(0)
    with pytest.raises(oracle.OracleError):
        HalosOracle(np.zeros(2, np.float32), [0]).gps_recv(0)


# ----------------------------------------------------------------------------------------------
# R5: merge special cases
# ----------------------------------------------------------------------------------------------
@pytest.mark.parametrize("dtype", [np.float32, np.float64])
def test_merge_special_cases(dtype):
    rng = np.random.default_rng(3)
    P = 64
    th_init = rng.normal(size=P).astype(np.float32)

    def run(alpha):
        o = HalosOracle(th_init, [0], K=2, alpha=alpha, dtype=dtype)
        for _ in range(2):
            s0 = o.buffer("th0", 0)
            o.arrive(0, (s0 + rng.normal(size=P).astype(np.float32) * np.float32(1e-2)).astype(np.float32))
        o.gps_recv(0)
        s0 = o.buffer("th0", 0)
        o.arrive(0, (s0 + np.float32(1e-2)).astype(np.float32))    # an update while Theta_i is in flight
        before = o.buffer("th", 0).copy()
        o.pull(0)
        return o, before

    o, before = run(0.0)
    np.testing.assert_array_equal(o.buffer("th", 0), before)        # alpha = 0: LPS isolated
    o, before = run(1.0)
    np.testing.assert_array_equal(o.buffer("th", 0), o.buffer("inbox", 0))   # alpha = 1: in-flight update discarded
    np.testing.assert_array_equal(o.buffer("anchor", 0), o.buffer("th", 0))
    o, before = run(0.25)
    ref = 0.75 * before.astype(np.float64) + 0.25 * o.buffer("inbox", 0).astype(np.float64)
    np.testing.assert_allclose(o.buffer("th", 0), ref, rtol=3e-7 if dtype == np.float32 else 1e-15)


# ----------------------------------------------------------------------------------------------
# R8: independent history-indexed interpreter on random legal traces
# ----------------------------------------------------------------------------------------------
@pytest.mark.parametrize("seed", range(6))
def test_random_traces_against_paper_interpreter(seed):
    rng = np.random.default_rng(100 + seed)
    P = 5
    worker_lps = [[0, 0, 1], [0, 1, 1, 2], [0, 0, 0], [0, 1], [0, 1, 2, 2, 1, 0], [0]][seed]
    K = [2, 3, 1, 4, 2, 1][seed]
    hp = dict(eta_l=float(rng.uniform(0.05, 1)), beta_l=float(rng.uniform(0, 0.95)),
              eta_g=float(rng.uniform(0.05, 1)), beta_g=float(rng.uniform(0, 0.95)), alpha=float(rng.uniform(0, 1)))
    th_init = rng.normal(size=P).astype(np.float32)
    o = HalosOracle(th_init, worker_lps, K=K, dtype=np.float64, **hp)
    it = PaperInterpreter([float(x) for x in th_init], worker_lps, hp["eta_l"], hp["beta_l"], hp["eta_g"],
                          hp["beta_g"], hp["alpha"], K, zero=0.0)
    events = tr.random_trace(worker_lps, 120, K, seed)
    assert {int(k) for k in events["kind"]} == {tr.ARRIVE, tr.GPS_RECV, tr.PULL}
    for ev in events:
        kind, l, w = int(ev["kind"]), int(ev["lps"]), int(ev["worker"])
        if kind == tr.ARRIVE:
            # the interpreter's worker snapshot is exact double; the oracle's is rounded to fp32.
            # Feed both the same *displacement*: each gets its own start + noise.
            noise = rng.normal(size=P) * 0.05
            s0 = o.buffer("th0", w).astype(np.float64)
            thH = (s0 + noise).astype(np.float32)
            fed = thH.astype(np.float64) - s0
            p1 = o.arrive(w, thH)
            p2 = it.arrive(w, [a + b for a, b in zip(it.start[w], fed)])
            assert p1 == p2
        elif kind == tr.GPS_RECV:
            o.gps_recv(l)
            it.gps_recv(l)
        else:
            o.pull(l)
            it.pull(l)
        for ll in range(max(worker_lps) + 1):
            np.testing.assert_allclose(o.buffer("th", ll), it.lps_model(ll), rtol=1e-11, atol=1e-13)
            assert o.counters(ll)["t"] == it.t[ll] and o.counters(ll)["t_last"] == it.t_last[ll]
        np.testing.assert_allclose(o.buffer("Theta"), it.gps_model(), rtol=1e-11, atol=1e-13)
        assert o.counters(0)["i"] == len(it.Theta) - 1


# ----------------------------------------------------------------------------------------------
# R6: invariants of an elementwise method
# ----------------------------------------------------------------------------------------------
def _replay(o, events, make_result):
    for ev in events:
        kind, l, w = int(ev["kind"]), int(ev["lps"]), int(ev["worker"])
        if kind == tr.ARRIVE:
            o.arrive(w, make_result(o, w))
        elif kind == tr.GPS_RECV:
            o.gps_recv(l)
        else:
            o.pull(l)


def test_slicing_permutation_and_scaling_invariance():
    from paper_2506_04531_b200.inputs import gen
    from paper_2506_04531_b200.inputs.layouts import flat_layout
    P = 4096
    lay = flat_layout("x", P)
    worker_lps = [0, 0, 1, 1]
    events = tr.random_trace(worker_lps, 150, 4, 42)
    init = gen.theta_init(lay, 9)

    def run(lo, hi, perm=None, scale=1.0, zero_init=False):
        base = np.zeros(hi - lo, np.float32) if zero_init else init[lo:hi]
        if perm is not None:
            base = base[perm]
        o = HalosOracle(base, worker_lps, K=4, dtype=np.float32)

        def mk(o, w):
            r = o.worker_info(w)["round"]
            z = gen.unit_noise(gen.stream_key(9, gen.STREAM_WORKER + w, r), lo, hi) * np.float32(1e-3 * scale)
            if perm is not None:
                z = z[perm]
            return o.buffer("th0", w) + z
        _replay(o, events, mk)
        return o

    full = run(0, P)
    part = run(1000, 1777)
    for name, idx in [("Theta", 0), ("Mg", 0), ("th", 0), ("th", 1), ("ml", 1), ("anchor", 0), ("outbox", 1),
                      ("inbox", 0), ("th0", 3)]:
        np.testing.assert_array_equal(full.buffer(name, idx)[1000:1777], part.buffer(name, idx))
    perm = np.random.default_rng(0).permutation(P)
    pm = run(0, P, perm=perm)
    np.testing.assert_array_equal(full.buffer("Theta")[perm], pm.buffer("Theta"))
    np.testing.assert_array_equal(full.buffer("th", 1)[perm], pm.buffer("th", 1))
    # all models start at zero: scaling every displacement by 2^k scales the whole state exactly
    a = run(0, 512, zero_init=True)
    b = run(0, 512, zero_init=True, scale=8.0)
    np.testing.assert_array_equal(a.buffer("Theta") * np.float32(8), b.buffer("Theta"))
    np.testing.assert_array_equal(a.buffer("ml", 0) * np.float32(8), b.buffer("ml", 0))
    # counters: i counts GPS_RECV events, t counts arrivals per LPS
    assert full.counters(0)["i"] == int((events["kind"] == tr.GPS_RECV).sum())
    for l in (0, 1):
        assert full.counters(l)["t"] == int(((events["kind"] == tr.ARRIVE) & (events["lps"] == l)).sum())


def test_float_and_double_oracles_agree_loosely():
    from paper_2506_04531_b200.inputs import gen
    from paper_2506_04531_b200.inputs.layouts import flat_layout
    P = 2048
    lay = flat_layout("x", P)
    worker_lps = [0, 0, 1, 1]
    events = tr.random_trace(worker_lps, 200, 8, 1)
    init = gen.theta_init(lay, 2)
    of = HalosOracle(init, worker_lps, K=8, dtype=np.float32)
    od = HalosOracle(init, worker_lps, K=8, dtype=np.float64)

    def mk(o, w):
        r = o.worker_info(w)["round"]
        return gen.worker_result(o.buffer("th0", w), lay, 2, w, r)
    _replay(of, events, mk)
    _replay(od, events, mk)
    for name, idx in [("Theta", 0), ("th", 0), ("th", 1)]:
        a, b = of.buffer(name, idx).astype(np.float64), od.buffer(name, idx)
        assert np.max(np.abs(a - b)) / np.sqrt(np.mean(b * b)) < 2e-5


# ----------------------------------------------------------------------------------------------
# bf16 worker copies: round-to-nearest-even, pinned to the definition and to a library routine
# ----------------------------------------------------------------------------------------------
def _rne_by_definition(x: float) -> int:
    """Nearest bf16 to x by exact comparison of the two neighbours; ties to even mantissa."""
    u = struct.unpack("<I", struct.pack("<f", x))[0]
    lo = u & 0xFFFF0000
    if lo == u:
        return u >> 16
    hi = lo + 0x10000   # next bf16 pattern away from zero (same sign bit); exact also across binades
    f = lambda b: Fr(struct.unpack("<f", struct.pack("<I", b))[0])
    if (hi & 0x7F800000) == 0x7F800000:   # would round to infinity: compare with 2^128 in exact arithmetic
        sign = -1 if (u >> 31) else 1
        v_hi = sign * Fr(2) ** 128
    else:
        v_hi = f(hi)
    dl, dh = abs(Fr(x) - f(lo)), abs(v_hi - Fr(x))
    if dl < dh:
        return lo >> 16
    if dh < dl:
        return hi >> 16
    return (lo >> 16) if ((lo >> 16) & 1) == 0 else (hi >> 16)


def test_bf16_rounding_brute_force():
    import torch
    rng = np.random.default_rng(0)
    pats = []
    for upper in [0x0000, 0x0001, 0x007F, 0x0080, 0x3F80, 0x3F81, 0x3FFF, 0x407F, 0x7F7E, 0x7F7F, 0x00FF, 0x1234]:
        for lower in [0x0000, 0x0001, 0x7FFF, 0x8000, 0x8001, 0xFFFF, 0x4000, 0xC000]:
            for sign in (0, 1):
                pats.append((sign << 31) | (upper << 16) | lower)
    pats += [int(x) for x in rng.integers(0, 1 << 32, size=3000, dtype=np.uint64)]
    arr = np.array(pats, dtype=np.uint32).view(np.float32)
    arr = arr[np.isfinite(arr)]
    got = np.array([oracle.f32_to_bf16(float(x)) for x in arr], dtype=np.uint16)
    want = np.array([_rne_by_definition(float(x)) for x in arr], dtype=np.uint16)
    np.testing.assert_array_equal(got, want)
    lib = torch.from_numpy(arr.copy()).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    np.testing.assert_array_equal(got, lib)
    for h in [0x0000, 0x3F80, 0xBF80, 0x0001, 0x7F7F, 0x8000]:
        assert oracle.f32_to_bf16(oracle.bf16_to_f32(h)) == h       # widening is exact


def test_bf16_worker_snapshots():
    rng = np.random.default_rng(2)
    P = 256
    th_init = rng.normal(size=P).astype(np.float32) * np.float32(0.02)
    o = HalosOracle(th_init, [0, 0], K=3, worker_dtype=oracle.BF16, dtype=np.float32)
    import torch
    to_bf16 = lambda x: torch.from_numpy(np.ascontiguousarray(x, np.float32)).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    widen = lambda h: (h.astype(np.uint32) << 16).view(np.float32)
    np.testing.assert_array_equal(o.buffer("th0", 1), to_bf16(th_init))
    s0 = o.buffer("th0", 0).copy()
    thH = to_bf16(widen(s0) + rng.normal(size=P).astype(np.float32) * np.float32(1e-3))
    th_before, m_before = o.buffer("th", 0).copy(), o.buffer("ml", 0).copy()
    o.arrive(0, thH)
    # delta is formed from the ROUNDED stored values; the snapshot is the rounded new model
    d = widen(thH).astype(np.float64) - widen(s0).astype(np.float64)
    m = 0.9 * m_before + d
    ref = th_before + np.float32(0.2).astype(np.float64) * ((1 - np.float32(0.9).astype(np.float64)) * d + np.float32(0.9).astype(np.float64) * m)
    np.testing.assert_allclose(o.buffer("th", 0), ref, rtol=2e-7, atol=1e-9)
    np.testing.assert_array_equal(o.buffer("th0", 0), to_bf16(o.buffer("th", 0)))
    np.testing.assert_array_equal(o.buffer("th0", 1), to_bf16(th_init))      # the other worker keeps its stale start


# ----------------------------------------------------------------------------------------------
# Bookkeeping: the worker's staleness (LPS updates applied since it was last scheduled, Alg. 1
# lines 10 and 12: the worker is handed theta_t right after update t) counted from the trace alone
# ----------------------------------------------------------------------------------------------
def _staleness_from_trace(events):
    """For every ARRIVE: how many arrivals its LPS processed after this worker's previous arrival
    (all earlier ones for a first arrival: every worker starts from the initial model, t = 0)."""
    out = []
    for n, ev in enumerate(events):
        if int(ev["kind"]) != tr.ARRIVE:
            continue
        l, w = int(ev["lps"]), int(ev["worker"])
        prev = max([k for k in range(n) if int(events[k]["kind"]) == tr.ARRIVE and int(events[k]["worker"]) == w], default=-1)
        out.append(sum(1 for k in range(prev + 1, n) if int(events[k]["kind"]) == tr.ARRIVE and int(events[k]["lps"]) == l))
    return out


def test_worker_staleness_bookkeeping():
    # the worked 12-event example: arrivals A0 A2 A1 A0 . A2 . . A1 . A0 with w0, w1 at LPS 0 and w2 at LPS 1
    worker_lps = [0, 0, 1]
    ev = np.zeros(12, dtype=tr.EVENT_DTYPE)
    for n, tok in enumerate(_TRACE_R7):
        kind = {"A": tr.ARRIVE, "G": tr.GPS_RECV, "P": tr.PULL}[tok[0]]
        ev[n]["kind"] = kind
        ev[n]["worker"] = int(tok[1]) if kind == tr.ARRIVE else 0
        ev[n]["lps"] = worker_lps[int(tok[1])] if kind == tr.ARRIVE else int(tok[1])
    assert _staleness_from_trace(ev) == [0, 0, 1, 1, 0, 1, 1]          # by hand from the order above
    cases = [(ev, worker_lps, 2)]
    for seed, wl, K in ((3, [0, 0, 0, 1, 1], 3), (4, [0, 1, 2, 2, 1, 0, 0], 2)):
        cases.append((tr.random_trace(wl, 150, K, seed), wl, K))
    wl = [0, 0, 0, 1, 1, 1]
    cases.append((tr.generate_trace(tr.TraceSpec(P=1000, worker_lps=wl, speeds=[1, 1.3, 3.7, 2, 2.2, 4], t_profiled_ms=1.0,
                                                 n_arrivals=120, K=5)), wl, 5))
    for events, wl, K in cases:
        o = HalosOracle(np.zeros(3, np.float32), wl, K=K)
        got = []
        for e in events:
            kind, l, w = int(e["kind"]), int(e["lps"]), int(e["worker"])
            if kind == tr.ARRIVE:
                got.append(o.counters(l)["t"] - o.worker_info(w)["sched_t"])
                o.arrive(w, np.zeros(3, np.float32))
                assert o.worker_info(w)["sched_t"] == o.counters(l)["t"]
            elif kind == tr.GPS_RECV:
                o.gps_recv(l)
            else:
                o.pull(l)
        assert got == _staleness_from_trace(events)
        assert [o.worker_info(w)["round"] for w in range(len(wl))] == \
            [int(((events["kind"] == tr.ARRIVE) & (events["worker"] == w)).sum()) for w in range(len(wl))]
        o.close()


# ----------------------------------------------------------------------------------------------
# The event log (what the driver must report per event) derived from the oracle's counters, checked
# against a direct count over the trace, and the stored hashes of the configured traces' logs
# ----------------------------------------------------------------------------------------------
def test_event_log_bookkeeping_and_golden_hashes():
    from paper_2506_04531_b200.inputs import workloads
    from sliced_oracle import log_hash, oracle_event_log
    wl = workloads.workload("toy_k4")
    ev = wl.trace()
    log = oracle_event_log(wl, ev)
    kind, lps = ev["kind"], ev["lps"]
    t = [0] * wl.n_lps
    t_last = [0] * wl.n_lps
    answered_at = [0] * wl.n_lps
    i = 0
    for k in range(len(ev)):
        l = int(lps[k])
        if kind[k] == tr.ARRIVE:
            t[l] += 1
            assert int(log["pushed"][k]) == int(t[l] - t_last[l] == wl.K)       # Alg. 1 line 13
        elif kind[k] == tr.GPS_RECV:
            i += 1
            answered_at[l] = i
        else:
            assert int(log["gps_lag"][k]) == i - answered_at[l]                 # GPS iterations since its Theta_i
            t_last[l] = t[l]                                                     # line 18
        assert (int(log["t"][k]), int(log["t_last"][k]), int(log["gps_iter"][k])) == (t[l], t_last[l], i)
    assert int(log["pushed"].sum()) >= 20 and int(log["gps_lag"].max()) >= 1
    golden = {}
    for line in (Path(__file__).parent / "golden" / "event_log_hashes.txt").read_text().splitlines():
        if line and not line.startswith("#"):
            name, n, digest = line.split()
            golden[name] = (int(n), digest)
    assert set(golden) >= {"toy", "toy_k4", "70m", "160m", "410m"}
    for name in ("toy", "toy_k4", "70m", "410m"):
        w = workloads.workload(name)
        e = w.trace()
        assert (len(e), log_hash(oracle_event_log(w, e))) == golden[name], name
