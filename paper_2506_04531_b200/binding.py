"""Thin ctypes binding of the C ABI in include/halos.h -- argument marshalling only.

Every step of the update path runs in the CUDA library; PyTorch is used for device memory
(the allocator handed to ``halos_create``), streams and host<->device plumbing.  There is no CPU
path: if ``libhalos_b200.so`` is missing or no CUDA device is present, creating a context raises.
"""
from __future__ import annotations

import ctypes as C
from pathlib import Path
from typing import Callable, Optional, Sequence

import numpy as np

_PKG = Path(__file__).resolve().parent
LIB_PATH = _PKG / "libhalos_b200.so"

OK, ERR_INVALID_ARG, ERR_BAD_STATE, ERR_OOM, ERR_CUDA, ERR_UNSUPPORTED, ERR_TIMEOUT = range(7)
F32, BF16 = 0, 1
FLAG_STATS = 1
FLAG_MATERIALISE_DELTA = 2
FLAG_GUARD = 4
IDLE, PUSHED, ANSWERED = 0, 1, 2
BUF_THETA_G, BUF_M_G, BUF_THETA_L, BUF_M_L, BUF_ANCHOR, BUF_OUTBOX, BUF_INBOX, BUF_THETA0, BUF_ACC_L, BUF_ACC_G = range(10)
OPT_PAPER, OPT_DELAYED_NESTEROV = 0, 1
EV_ARRIVE, EV_GPS_RECV, EV_PULL = 0, 1, 2
K_ARRIVE, K_ARRIVE_PUSH, K_PUSH, K_GPS, K_PULL, K_ARRIVE_MULTI, K_GPS_PULL = range(7)
KERNEL_NAMES = ("arrive", "arrive_push", "push", "gps", "pull", "arrive_multi", "gps_pull")

EXPORTED = (
    "halos_default_config", "halos_create", "halos_worker_delta", "halos_worker_delta_host", "halos_lps_apply",
    "halos_lps_push", "halos_gps_merge", "halos_lps_pull", "halos_destroy", "halos_replay", "halos_peek",
    "halos_read", "halos_counters", "halos_worker_info", "halos_stats", "halos_info", "halos_timing_enable",
    "halos_timing_read", "halos_strerror", "halos_last_error", "halos_push_noalloc", "halos_export_file",
    "halos_import_file", "halos_replay_batched", "halos_batch_info", "halos_check_guards", "halos_replay_stream",
    "halos_flush", "halos_gps_merge_pull", "halos_stats_log", "halos_worker_fetch_host", "halos_fetch_sync",
    "halos_timing_launches", "halos_replay_results",
)
NOALLOC_MAX_ELEMS = 1 << 29

ALLOC_FN = C.CFUNCTYPE(C.c_void_p, C.c_size_t, C.c_void_p)
FREE_FN = C.CFUNCTYPE(None, C.c_void_p, C.c_void_p)
PRODUCER_FN = C.CFUNCTYPE(C.c_int, C.c_void_p, C.c_uint32, C.c_uint32, C.c_uint64,
                          C.POINTER(C.c_void_p), C.POINTER(C.POINTER(C.c_void_p)))


class Config(C.Structure):
    _fields_ = [
        ("struct_size", C.c_uint32), ("n_lps", C.c_uint32), ("n_workers", C.c_uint32),
        ("worker_lps", C.POINTER(C.c_uint32)), ("n_tensors", C.c_uint32),
        ("tensor_numel", C.POINTER(C.c_uint64)),
        ("eta_l", C.c_float), ("beta_l", C.c_float), ("eta_g", C.c_float), ("beta_g", C.c_float),
        ("alpha", C.c_float), ("K", C.c_uint32), ("worker_dtype", C.c_uint32), ("flags", C.c_uint32),
        ("device", C.c_int32), ("stream", C.c_void_p),
        ("alloc", ALLOC_FN), ("free_", FREE_FN), ("alloc_user", C.c_void_p),
        ("chunk_elems", C.c_uint32), ("optimizer", C.c_uint32), ("delay_l", C.c_uint32), ("delay_g", C.c_uint32),
        ("reserved", C.c_uint32),
    ]


class Event(C.Structure):
    _fields_ = [("kind", C.c_uint8), ("lps", C.c_uint8), ("worker", C.c_uint16), ("pad", C.c_uint32),
                ("time_ns", C.c_int64)]


LAUNCH_RECORD_DTYPE = np.dtype([("kind", np.uint32), ("events", np.uint32), ("bytes_per_param", np.uint32), ("ms", np.float32)])

EVENT_LOG_DTYPE = np.dtype([
    ("index", np.uint32), ("kind", np.uint8), ("lps", np.uint8), ("worker", np.uint16),
    ("t", np.uint64), ("t_last", np.uint64), ("gps_iter", np.uint64), ("worker_staleness", np.uint64),
    ("gps_lag", np.uint64), ("pushed", np.uint8), ("fused", np.uint8), ("pad", np.uint8, (6,))])


class HalosError(RuntimeError):
    def __init__(self, status: int, message: str):
        super().__init__(f"halos status {status}: {message}")
        self.status = status


_lib = None


def load_library():
    """Loads libhalos_b200.so (built in-tree by ``paper_2506_04531_b200.build``); raises if absent."""
    global _lib
    if _lib is not None:
        return _lib
    if not LIB_PATH.exists():
        raise FileNotFoundError(
            f"{LIB_PATH} is missing: build it with `python -m paper_2506_04531_b200.build` (there is no fallback path)")
    lib = C.CDLL(str(LIB_PATH))
    vp, u32, u64, i32 = C.c_void_p, C.c_uint32, C.c_uint64, C.c_int
    lib.halos_default_config.argtypes = [C.POINTER(Config)]
    lib.halos_default_config.restype = None
    lib.halos_create.argtypes = [C.POINTER(Config), vp, C.POINTER(vp)]
    lib.halos_worker_delta.argtypes = [vp, u32, vp, vp]
    lib.halos_worker_delta_host.argtypes = [vp, u32, vp]
    lib.halos_lps_apply.argtypes = [vp, u32, u32, C.POINTER(i32)]
    lib.halos_lps_push.argtypes = [vp, u32]
    lib.halos_gps_merge.argtypes = [vp, u32]
    lib.halos_lps_pull.argtypes = [vp, u32]
    lib.halos_gps_merge_pull.argtypes = [vp, u32]
    lib.halos_stats_log.argtypes = [vp, vp, u64]
    lib.halos_worker_fetch_host.argtypes = [vp, u32, vp]
    lib.halos_fetch_sync.argtypes = [vp]
    lib.halos_timing_launches.argtypes = [vp, vp, u64, C.POINTER(u64)]
    lib.halos_destroy.argtypes = [vp]
    lib.halos_replay.argtypes = [vp, vp, u32, PRODUCER_FN, vp, vp, C.POINTER(u32)]
    lib.halos_replay_batched.argtypes = [vp, vp, u32, PRODUCER_FN, vp, vp, C.POINTER(u32), u32]
    lib.halos_check_guards.argtypes = [vp, C.POINTER(C.c_int32)]
    lib.halos_replay_stream.argtypes = [vp, vp, u32, PRODUCER_FN, vp, vp, C.POINTER(u32), u32]
    lib.halos_flush.argtypes = [vp]
    lib.halos_replay_results.argtypes = [vp, vp, u32, vp, vp, C.POINTER(u32), u32, i32]
    lib.halos_batch_info.argtypes = [vp, C.POINTER(u64), C.POINTER(u64)]
    lib.halos_peek.argtypes = [vp, u32, u32, C.POINTER(vp), C.POINTER(u64)]
    lib.halos_read.argtypes = [vp, u32, u32, u64, u64, vp]
    lib.halos_counters.argtypes = [vp, u32, vp]
    lib.halos_worker_info.argtypes = [vp, u32, vp]
    lib.halos_stats.argtypes = [vp, u32, u32, vp]
    lib.halos_info.argtypes = [vp, C.POINTER(u64), C.POINTER(u32), C.POINTER(u32), C.POINTER(u64)]
    lib.halos_timing_enable.argtypes = [vp, i32]
    lib.halos_timing_read.argtypes = [vp, u32, C.POINTER(u64), C.POINTER(C.c_double)]
    lib.halos_export_file.argtypes = [vp, C.c_char_p]
    lib.halos_import_file.argtypes = [vp, C.c_char_p]
    lib.halos_push_noalloc.argtypes = [C.c_int32, vp, vp, vp, vp, u64, vp]
    lib.halos_strerror.argtypes = [i32]
    lib.halos_strerror.restype = C.c_char_p
    lib.halos_last_error.argtypes = [vp]
    lib.halos_last_error.restype = C.c_char_p
    for name in EXPORTED:
        if name not in ("halos_default_config", "halos_strerror", "halos_last_error"):
            getattr(lib, name).restype = C.c_int
    _lib = lib
    return lib


def _ptr(x) -> Optional[int]:
    """Device/host address of a torch tensor, numpy array, int or None."""
    if x is None:
        return None
    if isinstance(x, int):
        return x
    if hasattr(x, "data_ptr"):
        return x.data_ptr()
    if isinstance(x, np.ndarray):
        return x.ctypes.data
    raise TypeError(type(x))


def push_noalloc(theta, anchor, Delta_out, sqnorm_out, n=None, stream=None) -> int:
    """Delta_out = theta - anchor and sqnorm_out[0] = sum Delta^2 without any allocation by the library.

    For callers that cannot allocate device memory (frozen or full pools, no-cudaMalloc policies):
    all four tensors are the caller's (fp32 CUDA tensors / raw addresses, sqnorm_out one float64).
    Returns the status code instead of raising so that the size limit (NOALLOC_MAX_ELEMS ->
    ERR_UNSUPPORTED) can be handled by the caller.  Calls share one fixed scratch array inside the
    library: do not let two of them overlap on the GPU."""
    import torch
    lib = load_library()
    n = int(theta.numel()) if n is None else int(n)
    dev = theta.device.index if hasattr(theta, "device") and theta.device.index is not None else torch.cuda.current_device()
    st = (stream if stream is not None else torch.cuda.current_stream(dev)).cuda_stream
    return int(lib.halos_push_noalloc(dev, st, _ptr(theta), _ptr(anchor), _ptr(Delta_out), n, _ptr(sqnorm_out)))


def result_table(events: np.ndarray, results):
    """The pointer table halos_replay_results takes: entry k = address of results[k] for ARRIVE events, NULL otherwise.
    Build it once for a window that is replayed through ``Halos.replay_results`` (keep the tensors alive yourself)."""
    return (C.c_void_p * len(events))(*[(_ptr(r) if int(k) == EV_ARRIVE else None) for r, k in zip(results, events["kind"])])


class Halos:
    """A HALoS server-side context on one GPU (see include/halos.h for the meaning of every call).

    ``theta_init`` is a flat fp32 CUDA tensor of P elements; ``tensor_numel`` the tensor sizes of
    the layout (defaults to one tensor of P); device memory comes from the PyTorch caching
    allocator unless ``use_torch_allocator=False``; ``alloc_limit_bytes`` makes that allocator refuse
    requests beyond a budget (used to test the out-of-memory path).
    """

    def __init__(self, theta_init, worker_lps: Sequence[int], tensor_numel: Optional[Sequence[int]] = None, *,
                 n_lps: Optional[int] = None, eta_l=0.2, beta_l=0.9, eta_g=0.15, beta_g=0.5, alpha=0.25, K=32,
                 worker_dtype=F32, flags=0, chunk_elems=0, stream=None, use_torch_allocator=True,
                 alloc_limit_bytes: Optional[int] = None, optimizer=OPT_PAPER, delay_l=1, delay_g=1):
        import torch
        self._torch = torch
        if not torch.cuda.is_available():
            raise HalosError(ERR_CUDA, "no CUDA device: the update path has no CPU implementation")
        self._lib = load_library()
        if not (theta_init.is_cuda and theta_init.dtype == torch.float32 and theta_init.is_contiguous()):
            raise ValueError("theta_init must be a contiguous fp32 CUDA tensor")
        self.P = int(theta_init.numel())
        self.device = theta_init.device
        wl = np.ascontiguousarray(worker_lps, dtype=np.uint32)
        tn = np.ascontiguousarray(tensor_numel if tensor_numel is not None else [self.P], dtype=np.uint64)
        if int(tn.sum()) != self.P:
            raise ValueError("tensor sizes do not add up to theta_init.numel()")
        self.n_workers, self.n_tensors = int(wl.size), int(tn.size)
        self.n_lps = int(n_lps if n_lps is not None else wl.max() + 1)
        self.worker_lps = wl
        self.tensor_numel = tn
        self.tensor_off = np.concatenate([[0], np.cumsum(tn)]).astype(np.uint64)
        self.worker_dtype = int(worker_dtype)
        self.K = int(K)
        self._blocks = {}
        self._stream = stream if stream is not None else torch.cuda.current_stream(self.device)

        self._allocated = 0

        def _alloc(nbytes, _user):
            if alloc_limit_bytes is not None and self._allocated + int(nbytes) > alloc_limit_bytes:
                return None          # lets tests exercise the library's out-of-memory path
            self._allocated += int(nbytes)
            try:
                with torch.cuda.device(self.device):
                    t = torch.empty(int(nbytes), dtype=torch.uint8, device=self.device)
            except Exception:
                return None
            self._blocks[t.data_ptr()] = t
            return t.data_ptr()

        def _free(ptr, _user):
            self._blocks.pop(ptr, None)

        self._alloc_cb, self._free_cb = ALLOC_FN(_alloc), FREE_FN(_free)
        cfg = Config()
        self._lib.halos_default_config(C.byref(cfg))
        cfg.n_lps, cfg.n_workers, cfg.n_tensors = self.n_lps, self.n_workers, self.n_tensors
        cfg.worker_lps = wl.ctypes.data_as(C.POINTER(C.c_uint32))
        cfg.tensor_numel = tn.ctypes.data_as(C.POINTER(C.c_uint64))
        cfg.eta_l, cfg.beta_l, cfg.eta_g, cfg.beta_g, cfg.alpha = eta_l, beta_l, eta_g, beta_g, alpha
        cfg.K, cfg.worker_dtype, cfg.flags, cfg.chunk_elems = int(K), self.worker_dtype, int(flags), int(chunk_elems)
        cfg.optimizer, cfg.delay_l, cfg.delay_g = int(optimizer), int(delay_l), int(delay_g)
        cfg.device = self.device.index if self.device.index is not None else torch.cuda.current_device()
        cfg.stream = self._stream.cuda_stream
        if use_torch_allocator:
            cfg.alloc, cfg.free_ = self._alloc_cb, self._free_cb
        self._h = C.c_void_p()
        rc = self._lib.halos_create(C.byref(cfg), theta_init.data_ptr(), C.byref(self._h))
        if rc != OK:
            raise HalosError(rc, self._lib.halos_last_error(None).decode())
        self._keep = {}
        self._stream_hold = {}

    # ------------------------------------------------------------------ plumbing
    def _mark_in_use(self, x):
        """Tells the caching allocator that a CUDA tensor is read by work on the context's stream."""
        if hasattr(x, "record_stream") and getattr(x, "is_cuda", False):
            x.record_stream(self._stream)

    def _check(self, rc: int):
        if rc != OK:
            raise HalosError(rc, self._lib.halos_last_error(self._h).decode())

    def close(self):
        if getattr(self, "_h", None):
            self._lib.halos_destroy(self._h)
            self._h = None
            self._blocks.clear()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def __enter__(self):
        return self

    def __exit__(self, *exc):
        self.close()

    # ------------------------------------------------------------------ the seven calls
    def worker_delta(self, worker: int, thetaH=None, thetaH_ptrs: Optional[Sequence] = None):
        """thetaH: flat CUDA tensor (fp32, or bf16/int16/uint16 for bf16 copies) or raw address;
        thetaH_ptrs: one CUDA tensor (or address) per layout tensor."""
        if thetaH_ptrs is not None:
            arr = (C.c_void_p * self.n_tensors)(*[_ptr(t) for t in thetaH_ptrs])
            self._check(self._lib.halos_worker_delta(self._h, worker, None, arr))
            self._keep[worker] = (thetaH_ptrs, arr)      # borrowed until the apply: keep the tensors alive
        else:
            self._check(self._lib.halos_worker_delta(self._h, worker, _ptr(thetaH), None))
            self._keep[worker] = thetaH

    def worker_delta_host(self, worker: int, thetaH_host):
        """thetaH_host: flat host tensor/array in the worker dtype (pinned memory makes the copy asynchronous)."""
        self._check(self._lib.halos_worker_delta_host(self._h, worker, _ptr(thetaH_host)))
        self._keep[worker] = thetaH_host

    def worker_fetch_host(self, worker: int, dst_host):
        """Copies the model the worker restarts from to a host tensor/array of the worker dtype (pinned memory makes
        it asynchronous); complete after fetch_sync()."""
        self._check(self._lib.halos_worker_fetch_host(self._h, worker, _ptr(dst_host)))
        self._fetch_keep = getattr(self, "_fetch_keep", [])
        self._fetch_keep.append(dst_host)

    def fetch_sync(self):
        self._check(self._lib.halos_fetch_sync(self._h))
        self._fetch_keep = []

    def lps_apply(self, lps: int, worker: int) -> bool:
        due = C.c_int(0)
        self._check(self._lib.halos_lps_apply(self._h, lps, worker, C.byref(due)))
        return bool(due.value)

    def lps_push(self, lps: int):
        self._check(self._lib.halos_lps_push(self._h, lps))

    def gps_merge(self, lps: int):
        self._check(self._lib.halos_gps_merge(self._h, lps))

    def lps_pull(self, lps: int):
        self._check(self._lib.halos_lps_pull(self._h, lps))

    def gps_merge_pull(self, lps: int):
        """gps_merge(lps) directly followed by lps_pull(lps), as one launch."""
        self._check(self._lib.halos_gps_merge_pull(self._h, lps))

    # ------------------------------------------------------------------ auxiliary
    def replay(self, events: np.ndarray, producer: Callable, want_log: bool = True, max_batch: int = 1,
               keep_queued: bool = False):
        """events: structured array (kind, lps, worker, pad, time_ns); producer(event_index, worker, round)
        returns a flat tensor/address or a list of per-tensor tensors.  max_batch > 1 turns on multi-event
        fusion (then a result must stay valid until the producer is called again for the same worker).
        keep_queued=True is the streaming form: arrivals still queued at the end stay queued for the next
        call (launch them with flush()).  Returns the event log."""
        ev = np.ascontiguousarray(events)
        assert ev.dtype.itemsize == C.sizeof(Event)
        log = np.zeros(len(ev), dtype=EVENT_LOG_DTYPE) if want_log else None
        # Results are borrowed by the library until the kernels that read them have run.  They are kept per
        # worker: a worker's entry is replaced at its next producer call (the library has launched its previous
        # arrival by then) and every tensor is marked as in use on the context's stream, so that the caching
        # allocator does not hand its block to another stream while an enqueued kernel still reads it.
        hold = self._stream_hold if keep_queued else {}
        err = []

        def _prod(_user, index, worker, rnd, flat_out, ptrs_out):
            try:
                r = producer(int(index), int(worker), int(rnd))
                if isinstance(r, (list, tuple)):
                    arr = (C.c_void_p * self.n_tensors)(*[_ptr(t) for t in r])
                    hold[worker] = (r, arr)
                    ptrs_out[0] = C.cast(arr, C.POINTER(C.c_void_p))
                    for t in r:
                        self._mark_in_use(t)
                else:
                    hold[worker] = r
                    flat_out[0] = _ptr(r)
                    self._mark_in_use(r)
                return 0
            except Exception as e:  # surfaced after the call returns
                err.append(e)
                return 1

        cb = PRODUCER_FN(_prod)
        failed = C.c_uint32(0)
        fn = self._lib.halos_replay_stream if keep_queued else self._lib.halos_replay_batched
        rc = fn(self._h, ev.ctypes.data, len(ev), cb, None,
                log.ctypes.data if log is not None else None, C.byref(failed), int(max_batch))
        if err:
            raise err[0]
        if rc != OK:
            raise HalosError(rc, f"event {failed.value}: " + self._lib.halos_last_error(self._h).decode())
        return log

    def replay_results(self, events: np.ndarray, results, want_log: bool = True, max_batch: int = 1,
                       keep_queued: bool = False):
        """replay() for results that already exist: ``results[k]`` is the flat CUDA tensor (or address) of event k if
        it is an ARRIVE (anything else is ignored there).  No Python code runs per event.  The tensors must stay
        alive and unchanged until their kernels have run (with keep_queued: until flush())."""
        ev = np.ascontiguousarray(events)
        assert ev.dtype.itemsize == C.sizeof(Event) and len(results) == len(ev)
        table = results if isinstance(results, C.Array) else result_table(ev, results)
        log = np.zeros(len(ev), dtype=EVENT_LOG_DTYPE) if want_log else None
        failed = C.c_uint32(0)
        rc = self._lib.halos_replay_results(self._h, ev.ctypes.data, len(ev), table,
                                            log.ctypes.data if log is not None else None, C.byref(failed), int(max_batch),
                                            int(bool(keep_queued)))
        if rc != OK:
            raise HalosError(rc, f"event {failed.value}: " + self._lib.halos_last_error(self._h).decode())
        return log

    def flush(self):
        """Launches the arrivals that replay(..., keep_queued=True) left queued."""
        self._check(self._lib.halos_flush(self._h))
        self._stream_hold.clear()

    def peek(self, which: int, index: int = 0):
        """Zero-copy torch view of a state buffer (fp32, or int16 bit patterns for bf16 worker snapshots)."""
        torch = self._torch
        p, n = C.c_void_p(), C.c_uint64()
        self._check(self._lib.halos_peek(self._h, which, index, C.byref(p), C.byref(n)))
        bf = which == BUF_THETA0 and self.worker_dtype == BF16
        nbytes = n.value * (2 if bf else 4)
        iface = {"shape": (nbytes,), "typestr": "|u1", "data": (p.value, False), "version": 2}
        holder = type("_DevMem", (), {"__cuda_array_interface__": iface})()
        t = torch.as_tensor(holder, device=self.device)
        return t.view(torch.int16 if bf else torch.float32)

    def read(self, which: int, index: int = 0, offset: int = 0, count: Optional[int] = None) -> np.ndarray:
        count = self.P - offset if count is None else count
        bf = which == BUF_THETA0 and self.worker_dtype == BF16
        out = np.empty(count, dtype=np.uint16 if bf else np.float32)
        self._check(self._lib.halos_read(self._h, which, index, offset, count, out.ctypes.data))
        return out

    def counters(self, lps: int) -> dict:
        out = (C.c_uint64 * 5)()
        self._check(self._lib.halos_counters(self._h, lps, out))
        return {"t": out[0], "t_last": out[1], "phase": out[2], "t_push": out[3], "i": out[4]}

    def worker_info(self, worker: int) -> dict:
        out = (C.c_uint64 * 3)()
        self._check(self._lib.halos_worker_info(self._h, worker, out))
        return {"round": out[0], "sched_t": out[1], "pending": bool(out[2])}

    def stats(self, what: int, lps: int) -> np.ndarray:
        out = np.empty(self.n_tensors, dtype=np.float64)
        self._check(self._lib.halos_stats(self._h, what, lps, out.ctypes.data))
        return out

    def stats_log(self, log=None):
        """Attaches a float64 CUDA tensor of shape (records, 3, n_tensors) as the per-arrival statistics log
        (None detaches); the tensor is kept alive until it is replaced."""
        if log is None:
            self._check(self._lib.halos_stats_log(self._h, None, 0))
        else:
            assert log.is_cuda and log.is_contiguous() and log.dim() == 3 and tuple(log.shape[1:]) == (3, self.n_tensors)
            self._check(self._lib.halos_stats_log(self._h, log.data_ptr(), int(log.shape[0])))
        self._stats_log = log

    def info(self) -> dict:
        P, nt, nc, nl = C.c_uint64(), C.c_uint32(), C.c_uint32(), C.c_uint64()
        self._check(self._lib.halos_info(self._h, C.byref(P), C.byref(nt), C.byref(nc), C.byref(nl)))
        return {"P": P.value, "n_tensors": nt.value, "n_chunks": nc.value, "launches": nl.value}

    def export_file(self, path):
        self._check(self._lib.halos_export_file(self._h, str(path).encode()))

    def import_file(self, path):
        self._check(self._lib.halos_import_file(self._h, str(path).encode()))

    def check_guards(self) -> int:
        """-1 if every canary zone is intact, else the index of the first damaged buffer (FLAG_GUARD contexts)."""
        bad = C.c_int32(0)
        self._check(self._lib.halos_check_guards(self._h, C.byref(bad)))
        return int(bad.value)

    def batch_info(self) -> dict:
        a, b = C.c_uint64(), C.c_uint64()
        self._check(self._lib.halos_batch_info(self._h, C.byref(a), C.byref(b)))
        return {"multi_launches": a.value, "batched_arrivals": b.value}

    def timing_enable(self, on: bool = True):
        self._check(self._lib.halos_timing_enable(self._h, int(on)))

    def timing_launches(self) -> np.ndarray:
        """Per-launch records (kind, events, bytes_per_param, ms) of everything timed since timing_enable(True)."""
        n = C.c_uint64(0)
        self._check(self._lib.halos_timing_launches(self._h, None, 0, C.byref(n)))
        out = np.zeros(n.value, dtype=LAUNCH_RECORD_DTYPE)
        if n.value:
            self._check(self._lib.halos_timing_launches(self._h, out.ctypes.data, n.value, C.byref(n)))
        return out

    def timing_read(self) -> dict:
        out = {}
        for k, name in enumerate(KERNEL_NAMES):
            n, ms = C.c_uint64(), C.c_double()
            self._check(self._lib.halos_timing_read(self._h, k, C.byref(n), C.byref(ms)))
            out[name] = (n.value, ms.value)
        return out
