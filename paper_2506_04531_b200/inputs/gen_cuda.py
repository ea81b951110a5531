"""CUDA twin of gen.py: the same values, bit for bit, written straight into device memory.

Harness only (synthetic model initialisation and the stand-in for a worker's local training);
it is a separate shared library (libhalos_inputs.so) and not part of the update path.
"""
from __future__ import annotations

import ctypes as C
from pathlib import Path

import numpy as np

from . import gen
from .layouts import Layout

_LIB_PATH = Path(__file__).resolve().parent / "libhalos_inputs.so"
_lib = None


def _load():
    global _lib
    if _lib is None:
        if not _LIB_PATH.exists():
            raise FileNotFoundError(f"{_LIB_PATH} is missing: run `python -m paper_2506_04531_b200.build`")
        lib = C.CDLL(str(_LIB_PATH))
        lib.halos_synth_fill.argtypes = [C.c_void_p, C.c_void_p, C.c_int, C.c_void_p, C.c_void_p, C.c_void_p,
                                         C.c_uint32, C.c_uint64, C.c_uint64, C.c_uint64, C.c_void_p]
        lib.halos_synth_fill.restype = C.c_int
        _lib = lib
    return _lib


class DeviceGenerator:
    """Holds the per-tensor tables of one layout on the device."""

    def __init__(self, layout: Layout, seed: int, device="cuda", sigma_table=None):
        import torch
        self.torch = torch
        self.layout, self.seed, self.device = layout, int(seed), torch.device(device)
        base_t, sig_init = gen.init_tables(layout)
        sig_w = gen.worker_sigma_table(layout) if sigma_table is None else np.asarray(sigma_table, np.float32)
        dev = lambda a, dt: torch.from_numpy(np.ascontiguousarray(a).astype(dt)).to(self.device)
        self.base_t = dev(base_t, np.float32)
        self.sig_init = dev(sig_init, np.float32)
        self.sig_w = dev(sig_w, np.float32)
        self.off = dev(layout.offsets.astype(np.int64), np.int64)
        self.P = layout.P

    def _fill(self, out, src, dtype, base, sigma, key, lo, n):
        stream = self.torch.cuda.current_stream(self.device).cuda_stream
        rc = _load().halos_synth_fill(out.data_ptr(), src.data_ptr() if src is not None else None, dtype,
                                      base.data_ptr(), sigma.data_ptr(), self.off.data_ptr(),
                                      self.layout.n_tensors, key, lo, n, stream)
        if rc != 0:
            raise RuntimeError(f"halos_synth_fill: cudaError {rc}")
        return out

    def theta_init(self, lo: int = 0, hi: int | None = None):
        """Theta_0[lo:hi] as an fp32 CUDA tensor."""
        hi = self.P if hi is None else hi
        out = self.torch.empty(hi - lo, dtype=self.torch.float32, device=self.device)
        return self._fill(out, None, gen.F32, self.base_t, self.sig_init, gen.stream_key(self.seed, gen.STREAM_INIT, 0), lo, hi - lo)

    def worker_result(self, theta0, worker: int, rnd: int, out=None, worker_dtype: int = gen.F32, lo: int = 0):
        """theta_H = cast(widen(theta0) + sigma_k z) for global indices [lo, lo + theta0.numel())."""
        n = theta0.numel()
        if out is None:
            out = self.torch.empty_like(theta0)
        key = gen.stream_key(self.seed, gen.STREAM_WORKER + worker, rnd)
        return self._fill(out, theta0, worker_dtype, self.base_t, self.sig_w, key, lo, n)
