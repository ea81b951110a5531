"""C twin of gen.py (same values, bit for bit) for CPU runs over many millions of elements.

Harness only.  Built on demand with gcc next to its source; gen.py stays the definition and
tests/test_inputs.py checks that the two agree.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from pathlib import Path

import numpy as np

from . import gen
from .layouts import Layout

_HERE = Path(__file__).resolve().parent
_SRC = _HERE / "csrc" / "synth_inputs_cpu.c"
_LIB_PATH = _HERE / "libhalos_inputs_cpu.so"
_lib = None


_FLAGS_NOTE = _HERE / "libhalos_inputs_cpu.flags"


def _isa_flags():
    """-mavx2 where the host has it (the generator's inner loops vectorise; integer and separately rounded
    float operations give the same bits at any vector width)."""
    try:
        for line in open("/proc/cpuinfo"):
            if line.startswith("flags"):
                return ["-mavx2"] if "avx2" in line.split() else []
    except OSError:
        pass
    return []


def build(force: bool = False) -> Path:
    """Idempotent; rebuilt when the source is newer or when the library was built for instructions this host lacks."""
    isa = _isa_flags()
    if not force and _LIB_PATH.exists() and _LIB_PATH.stat().st_mtime >= _SRC.stat().st_mtime:
        built_with = _FLAGS_NOTE.read_text().split() if _FLAGS_NOTE.exists() else None
        if built_with is not None and set(built_with) <= set(isa):
            return _LIB_PATH
    tmp = _LIB_PATH.with_suffix(f".so.tmp{os.getpid()}")
    subprocess.run(["gcc", "-O3", *isa, "-ffp-contract=off", "-fno-fast-math", "-fPIC", "-shared", "-o", str(tmp), str(_SRC)],
                   check=True)
    os.replace(tmp, _LIB_PATH)
    _FLAGS_NOTE.write_text(" ".join(isa) + "\n")
    return _LIB_PATH


def _load():
    global _lib
    if _lib is None:
        lib = C.CDLL(str(build()))
        lib.halos_synth_fill_cpu.argtypes = [C.c_void_p, C.c_void_p, C.c_int, C.c_void_p, C.c_void_p, C.c_void_p,
                                             C.c_uint32, C.c_uint64, C.c_uint64, C.c_uint64]
        lib.halos_synth_fill_cpu.restype = None
        _lib = lib
    return _lib


class HostGenerator:
    """Per-layout tables plus the two generators of gen.py, computed by the C library."""

    def __init__(self, layout: Layout, seed: int, sigma_table=None):
        self.layout, self.seed = layout, int(seed)
        self.base_t, self.sig_init = (np.ascontiguousarray(a, np.float32) for a in gen.init_tables(layout))
        self.sig_w = np.ascontiguousarray(gen.worker_sigma_table(layout) if sigma_table is None else sigma_table, np.float32)
        self.off = np.ascontiguousarray(layout.offsets, np.uint64)

    def _fill(self, out, src, dtype, base, sigma, key, lo):
        _load().halos_synth_fill_cpu(out.ctypes.data, src.ctypes.data if src is not None else None, dtype,
                                     base.ctypes.data, sigma.ctypes.data, self.off.ctypes.data, self.layout.n_tensors,
                                     key, lo, out.size)
        return out

    def theta_init(self, lo: int = 0, hi: int | None = None) -> np.ndarray:
        hi = self.layout.P if hi is None else hi
        out = np.empty(hi - lo, np.float32)
        return self._fill(out, None, gen.F32, self.base_t, self.sig_init, gen.stream_key(self.seed, gen.STREAM_INIT, 0), lo)

    def worker_result(self, theta0: np.ndarray, worker: int, rnd: int, lo: int = 0, worker_dtype: int = gen.F32) -> np.ndarray:
        src = np.ascontiguousarray(theta0, np.float32 if worker_dtype == gen.F32 else np.uint16)
        out = np.empty_like(src)
        key = gen.stream_key(self.seed, gen.STREAM_WORKER + worker, rnd)
        return self._fill(out, src, worker_dtype, self.base_t, self.sig_w, key, lo)
