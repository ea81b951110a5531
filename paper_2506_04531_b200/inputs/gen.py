"""Seeded synthetic inputs (CPU / numpy side).

The update path only ever sees parameter-shaped arrays, so the paper's models and data are
replaced by a counter-based generator: every value is a pure function of
(seed, stream, round, global parameter index).  Index slices can therefore be generated
independently, which lets the CPU oracle replay a trace on a slice of a large model.

    key   = splitmix64-derived 64-bit key of (seed, stream, round)
    x     = key + index * 0x9E3779B97F4A7C15            (mod 2^64)
    h0,h1 = mix64(x), mix64(x ^ 0xD1B54A32D192ED03)      (splitmix64 finaliser)
    s     = sum of the eight 16-bit lanes of (h0, h1)    (Irwin-Hall, n = 8)
    z     = float32(s - 262140) * INV_STD                (unit variance, |z| <= 4.9)

Everything up to the last line is integer-exact and the last line is one rounded fp32
multiply, so the CUDA twin of this generator (gen_cuda.py) produces the same bits.

``theta_init`` and ``worker_result`` are the stand-ins for the model initialisation and for
a worker's H local training steps.  They contain none of the update rules.
"""
from __future__ import annotations

import numpy as np

from .layouts import Layout

F32, BF16 = 0, 1
_M64 = (1 << 64) - 1
GOLDEN = 0x9E3779B97F4A7C15
SALT1 = 0xD1B54A32D192ED03
INV_STD = np.float32(float.fromhex("0x1.3988e2p-16"))  # 1/sqrt(8 * (65536^2 - 1) / 12)
LANE_MEAN_SUM = 262140                                 # 8 * 32767.5

STREAM_INIT = 1
STREAM_WORKER = 1000  # + worker id


def _mix_int(z: int) -> int:
    z &= _M64
    z ^= z >> 30
    z = (z * 0xBF58476D1CE4E5B9) & _M64
    z ^= z >> 27
    z = (z * 0x94D049BB133111EB) & _M64
    z ^= z >> 31
    return z


def stream_key(seed: int, stream: int, rnd: int) -> int:
    """64-bit key of one noise stream; plain integer arithmetic, identical for both generators."""
    k = _mix_int((seed + GOLDEN) & _M64)
    k = _mix_int((k ^ ((stream + 1) * GOLDEN)) & _M64)
    k = _mix_int((k ^ ((rnd + 1) * SALT1)) & _M64)
    return k


def _mix_np(z: np.ndarray) -> np.ndarray:
    z = z ^ (z >> np.uint64(30))
    z = z * np.uint64(0xBF58476D1CE4E5B9)
    z = z ^ (z >> np.uint64(27))
    z = z * np.uint64(0x94D049BB133111EB)
    z = z ^ (z >> np.uint64(31))
    return z


def unit_noise(key: int, lo: int, hi: int) -> np.ndarray:
    """z for global indices [lo, hi): float32, mean 0, variance 1."""
    with np.errstate(over="ignore"):
        idx = np.arange(lo, hi, dtype=np.uint64)
        x = np.uint64(key) + idx * np.uint64(GOLDEN)
        h0 = _mix_np(x)
        h1 = _mix_np(x ^ np.uint64(SALT1))
    s = np.zeros(hi - lo, dtype=np.int64)
    for h in (h0, h1):
        for sh in (0, 16, 32, 48):
            s += ((h >> np.uint64(sh)) & np.uint64(0xFFFF)).astype(np.int64)
    return (s - LANE_MEAN_SUM).astype(np.float32) * INV_STD


def expand_per_tensor(layout: Layout, values: np.ndarray, lo: int, hi: int) -> np.ndarray:
    """values[k] repeated over the part of tensor k that falls inside [lo, hi)."""
    off = layout.offsets.astype(np.int64)
    out = np.empty(hi - lo, dtype=np.float32)
    k0 = int(np.searchsorted(off, lo, side="right") - 1)
    k = k0
    while k < layout.n_tensors and off[k] < hi:
        a, b = max(int(off[k]), lo), min(int(off[k + 1]), hi)
        if b > a:
            out[a - lo:b - lo] = values[k]
        k += 1
    return out


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round-to-nearest-even fp32 -> bf16 bit patterns (finite inputs)."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    bias = np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1))
    return ((u + bias) >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(h: np.ndarray) -> np.ndarray:
    return (np.ascontiguousarray(h, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def init_tables(layout: Layout):
    """(base, sigma) per tensor for Theta_0: matrices N(0, 0.02), norm weights 1, biases 0."""
    return layout.per_tensor(0.0, 1.0, 0.0), layout.per_tensor(0.02, 0.0, 0.0)


def worker_sigma_table(layout: Layout, sigma_matrix: float = 1e-3, sigma_vector: float = 1e-4):
    """Per-tensor scale of a worker's displacement: matrices 1e-3, 1-D tensors 1e-4."""
    return layout.per_tensor(sigma_matrix, sigma_vector, sigma_vector)


def theta_init(layout: Layout, seed: int, lo: int = 0, hi: int | None = None) -> np.ndarray:
    """Theta_0[lo:hi] as float32:  base_k + sigma_k * z."""
    hi = layout.P if hi is None else hi
    base_t, sigma_t = init_tables(layout)
    z = unit_noise(stream_key(seed, STREAM_INIT, 0), lo, hi)
    base = expand_per_tensor(layout, base_t, lo, hi)
    sigma = expand_per_tensor(layout, sigma_t, lo, hi)
    return base + sigma * z  # two separately rounded fp32 operations


def worker_result(theta0: np.ndarray, layout: Layout, seed: int, worker: int, rnd: int,
                  lo: int = 0, hi: int | None = None, worker_dtype: int = F32,
                  sigma_table: np.ndarray | None = None) -> np.ndarray:
    """Stand-in for H local training steps: theta_H = cast_w(widen(theta_0) + sigma_k * z).

    ``theta0`` is the worker's start snapshot restricted to [lo, hi) in the worker dtype
    (float32, or uint16 bf16 patterns); the result has the same dtype.
    """
    hi = layout.P if hi is None else hi
    if sigma_table is None:
        sigma_table = worker_sigma_table(layout)
    z = unit_noise(stream_key(seed, STREAM_WORKER + worker, rnd), lo, hi)
    sigma = expand_per_tensor(layout, sigma_table, lo, hi)
    if worker_dtype == F32:
        return np.ascontiguousarray(theta0, dtype=np.float32) + sigma * z
    wide = bf16_bits_to_f32(theta0)
    return f32_to_bf16_bits(wide + sigma * z)
