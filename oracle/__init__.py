"""CPU oracle for the HALoS update rules (Algorithm 1 + the ModelUpdate rule of Appendix E).

TEST INFRASTRUCTURE.  Only tests, the smoke check and the benchmark's CPU-baseline leg may
import this package; the CUDA library never does, and the two share no code.

The arithmetic lives in ``halos_oracle.hpp`` (plain sequential C++17).  This module builds it
with g++ (``-O2 -ffp-contract=off``, no fast-math) and wraps it with ctypes.  Buffers are
exposed as numpy views of the oracle's own storage.

Parity pins (tests/test_oracle_*.py): exact hand expansion in rational arithmetic on 8
parameters, the closed-form geometric momentum sum, reduction to plain local SGD and to
model averaging, window/merge special cases, an independently written history-indexed
interpreter on random traces, and bf16 rounding brute force.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from pathlib import Path

import numpy as np

_HERE = Path(__file__).resolve().parent
_LIB_PATH = _HERE / "libhalos_oracle.so"
_SOURCES = [_HERE / "halos_oracle_c.cpp", _HERE / "halos_oracle.hpp"]

F32, BF16 = 0, 1
IDLE, PUSHED, ANSWERED = 0, 1, 2
OPT_PAPER, OPT_DELAYED_NESTEROV = 0, 1
_WHICH = {"Theta": 0, "Mg": 1, "th": 2, "ml": 3, "anchor": 4, "outbox": 5, "inbox": 6, "th0": 7, "delta": 8, "acc": 9, "acc_g": 10}


def _cpu_has(flag: str) -> bool:
    try:
        for line in open("/proc/cpuinfo"):
            if line.startswith("flags"):
                return flag in line.split()
    except OSError:
        pass
    return False


def _isa_flags():
    """-mfma where the host has the instruction: std::fma then compiles to one vfmadd instead of a libm call
    (the same correctly rounded result, several times faster).  No other flag depends on the host."""
    return ["-mfma"] if _cpu_has("fma") else []


_FLAGS_NOTE = _HERE / "libhalos_oracle.flags"


def build(force: bool = False) -> Path:
    """Compile the oracle into a shared library next to its sources (idempotent).  The library is rebuilt
    when a source is newer or when it was built for instructions this host lacks."""
    isa = _isa_flags()
    if not force and _LIB_PATH.exists():
        newest = max(p.stat().st_mtime for p in _SOURCES)
        built_with = _FLAGS_NOTE.read_text().split() if _FLAGS_NOTE.exists() else None
        if _LIB_PATH.stat().st_mtime >= newest and built_with is not None and set(built_with) <= set(isa):
            return _LIB_PATH
    tmp = _LIB_PATH.with_suffix(f".so.tmp{os.getpid()}")
    cmd = ["g++", "-std=c++17", "-O2", "-ffp-contract=off", "-fno-fast-math", *isa, "-fPIC", "-shared",
           "-o", str(tmp), str(_SOURCES[0]), "-lpthread"]
    subprocess.run(cmd, check=True, cwd=str(_HERE))
    os.replace(tmp, _LIB_PATH)
    _FLAGS_NOTE.write_text(" ".join(isa) + "\n")
    return _LIB_PATH


_lib = None


def _load():
    global _lib
    if _lib is not None:
        return _lib
    lib = ctypes.CDLL(str(build()))
    c = ctypes
    lib.halos_oracle_create.restype = c.c_void_p
    lib.halos_oracle_create.argtypes = [c.c_int, c.c_uint64, c.c_uint32, c.c_uint32, c.c_void_p,
                                        c.c_double, c.c_double, c.c_double, c.c_double, c.c_double,
                                        c.c_uint32, c.c_int, c.c_void_p, c.c_int, c.c_uint32, c.c_uint32]
    lib.halos_oracle_destroy.argtypes = [c.c_void_p]
    lib.halos_oracle_error.restype = c.c_char_p
    lib.halos_oracle_error.argtypes = [c.c_void_p]
    lib.halos_oracle_arrive.argtypes = [c.c_void_p, c.c_uint32, c.c_void_p, c.POINTER(c.c_int)]
    lib.halos_oracle_gps_recv.argtypes = [c.c_void_p, c.c_uint32]
    lib.halos_oracle_push.argtypes = [c.c_void_p, c.c_uint32]
    lib.halos_oracle_pull.argtypes = [c.c_void_p, c.c_uint32]
    lib.halos_oracle_buffer.restype = c.c_void_p
    lib.halos_oracle_buffer.argtypes = [c.c_void_p, c.c_int, c.c_uint32]
    lib.halos_oracle_counters.argtypes = [c.c_void_p, c.c_uint32, c.c_void_p]
    lib.halos_oracle_worker.argtypes = [c.c_void_p, c.c_uint32, c.c_void_p]
    lib.halos_oracle_f32_to_bf16.restype = c.c_uint16
    lib.halos_oracle_f32_to_bf16.argtypes = [c.c_float]
    lib.halos_oracle_bf16_to_f32.restype = c.c_float
    lib.halos_oracle_bf16_to_f32.argtypes = [c.c_uint16]
    _lib = lib
    return lib


def f32_to_bf16(x: float) -> int:
    return int(_load().halos_oracle_f32_to_bf16(float(x)))


def bf16_to_f32(h: int) -> float:
    return float(_load().halos_oracle_bf16_to_f32(int(h)))


class OracleError(RuntimeError):
    pass


class HalosOracle:
    """One GPS, ``n_lps`` local parameter servers and ``n_workers`` workers over P parameters.

    ``dtype`` is the scalar type of the master state: ``np.float32`` (parity oracle) or
    ``np.float64`` (self-check oracle).  ``worker_dtype`` is F32 or BF16: the type worker
    snapshots theta_{t,0} are stored in and worker results theta_{t,H} are given in
    (bf16 as uint16 bit patterns).  ``optimizer=OPT_DELAYED_NESTEROV`` with ``delay_l/delay_g`` selects the
    delayed-Nesterov reading described in halos_oracle.hpp (then eta_l/eta_g are its unscaled rates).
    """

    def __init__(self, theta_init, worker_lps, *, n_lps=None, eta_l=0.2, beta_l=0.9, eta_g=0.15,
                 beta_g=0.5, alpha=0.25, K=32, worker_dtype=F32, dtype=np.float32,
                 optimizer=OPT_PAPER, delay_l=1, delay_g=1):
        lib = _load()
        theta_init = np.ascontiguousarray(theta_init, dtype=np.float32)
        wl = np.ascontiguousarray(worker_lps, dtype=np.uint32)
        self.P = int(theta_init.size)
        self.n_workers = int(wl.size)
        self.n_lps = int(n_lps if n_lps is not None else (wl.max() + 1))
        self.worker_lps = wl.copy()
        self.dtype = np.dtype(dtype)
        assert self.dtype in (np.dtype(np.float32), np.dtype(np.float64))
        self.worker_dtype = int(worker_dtype)
        self.K = int(K)
        self._lib = lib
        self._h = lib.halos_oracle_create(int(self.dtype == np.float64), self.P, self.n_lps,
                                          self.n_workers, wl.ctypes.data, float(eta_l), float(beta_l),
                                          float(eta_g), float(beta_g), float(alpha), int(K),
                                          self.worker_dtype, theta_init.ctypes.data, int(optimizer),
                                          int(delay_l), int(delay_g))
        if not self._h:
            raise OracleError("halos_oracle_create failed")

    def close(self):
        if getattr(self, "_h", None):
            self._lib.halos_oracle_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def _check(self, rc):
        if rc != 0:
            raise OracleError(self._lib.halos_oracle_error(self._h).decode())

    # --- events (Algorithm 1) -------------------------------------------------------------
    def arrive(self, worker: int, thetaH) -> bool:
        """Worker result theta_{t,H} arrives (lines 9-15, 25). Returns True if Delta was pushed."""
        want = np.float32 if self.worker_dtype == F32 else np.uint16
        a = np.ascontiguousarray(thetaH, dtype=want)
        if a.size != self.P:
            raise ValueError("thetaH has the wrong size")
        pushed = ctypes.c_int(0)
        self._check(self._lib.halos_oracle_arrive(self._h, int(worker), a.ctypes.data, ctypes.byref(pushed)))
        return bool(pushed.value)

    def push(self, lps: int) -> None:
        """Form Delta = theta_t - theta_{t_last} now (line 14), whatever the window counter says."""
        self._check(self._lib.halos_oracle_push(self._h, int(lps)))

    def gps_recv(self, lps: int) -> None:
        """The GPS receives Delta from this LPS and answers with Theta_i (lines 2-4)."""
        self._check(self._lib.halos_oracle_gps_recv(self._h, int(lps)))

    def pull(self, lps: int) -> None:
        """The LPS merges the Theta_i it was sent (lines 17-20)."""
        self._check(self._lib.halos_oracle_pull(self._h, int(lps)))

    # --- state ----------------------------------------------------------------------------
    def buffer(self, which: str, idx: int = 0) -> np.ndarray:
        """numpy view (no copy) of one state buffer: Theta, Mg, th, ml, anchor, outbox, inbox, th0, delta."""
        p = self._lib.halos_oracle_buffer(self._h, _WHICH[which], int(idx))
        if not p:
            raise IndexError(f"{which}[{idx}]")
        if which == "th0":
            ct, dt = (ctypes.c_float, np.float32) if self.worker_dtype == F32 else (ctypes.c_uint16, np.uint16)
        else:
            ct, dt = (ctypes.c_float, np.float32) if self.dtype == np.float32 else (ctypes.c_double, np.float64)
        arr = np.ctypeslib.as_array(ctypes.cast(p, ctypes.POINTER(ct)), shape=(self.P,))
        return arr.view(dt)

    def sq_norms(self, which: str, idx: int, offsets) -> np.ndarray:
        """Per-tensor sum of squares of a buffer, accumulated in fp64 (tensor k = [offsets[k], offsets[k+1]))."""
        x = self.buffer(which, idx).astype(np.float64)
        off = np.asarray(offsets, dtype=np.int64)
        return np.array([float(np.dot(x[a:b], x[a:b])) for a, b in zip(off[:-1], off[1:])])

    def counters(self, lps: int) -> dict:
        out = (ctypes.c_uint64 * 5)()
        self._lib.halos_oracle_counters(self._h, int(lps), out)
        return {"t": out[0], "t_last": out[1], "phase": out[2], "t_push": out[3], "i": out[4]}

    def worker_info(self, worker: int) -> dict:
        out = (ctypes.c_uint64 * 2)()
        self._lib.halos_oracle_worker(self._h, int(worker), out)
        return {"round": out[0], "sched_t": out[1]}
