"""CPU-side checks of the boundary: the shared library loads without a GPU, exports every symbol
that include/halos.h declares, the ctypes mirror of the structs matches the C layout, and calls
that can be judged without a device fail cleanly (no compute is attempted here)."""
from __future__ import annotations

import ctypes as C
import re
import subprocess
import sys
from pathlib import Path

import pytest

ROOT = Path(__file__).resolve().parent.parent
HEADER = ROOT / "include" / "halos.h"


@pytest.fixture(scope="module")
def lib():
    from paper_2506_04531_b200 import build
    build.build()
    from paper_2506_04531_b200 import binding
    return binding.load_library()


def _declared():
    text = re.sub(r"/\*.*?\*/", "", HEADER.read_text(), flags=re.S)
    names = set(re.findall(r"\b(halos_[a-z_0-9]+)\s*\(", text))
    return {n for n in names if not n.endswith("_fn")}


def test_every_declared_symbol_is_exported(lib):
    from paper_2506_04531_b200 import binding
    declared = _declared()
    core = {"halos_create", "halos_worker_delta", "halos_lps_apply", "halos_lps_push", "halos_gps_merge",
            "halos_lps_pull", "halos_destroy"}
    assert core <= declared
    for name in sorted(declared):
        assert hasattr(lib, name), f"{name} declared in halos.h but not exported"
    assert declared == set(binding.EXPORTED), declared ^ set(binding.EXPORTED)


def test_struct_layout_matches_c(tmp_path, lib):
    from paper_2506_04531_b200 import binding
    src = tmp_path / "layout.c"
    fields = [f[0] for f in binding.Config._fields_]
    lines = ['#include <stdio.h>', '#include <stddef.h>', '#include "halos.h"', "int main(void){",
             'printf("%zu\\n", sizeof(halos_config));']
    lines += [f'printf("%zu\\n", offsetof(halos_config, {f}));' for f in fields]
    lines += ['printf("%zu %zu\\n", sizeof(halos_event), sizeof(halos_event_log));',
              'printf("%zu %zu %zu\\n", offsetof(halos_event_log, t), offsetof(halos_event_log, gps_lag), offsetof(halos_event_log, pushed));',
              'printf("%zu %zu %zu %zu %zu\\n", sizeof(halos_launch_record), offsetof(halos_launch_record, kind), '
              'offsetof(halos_launch_record, events), offsetof(halos_launch_record, bytes_per_param), offsetof(halos_launch_record, ms));',
              'printf("%d %d\\n", (int)HALOS_K_COUNT, (int)HALOS_K_GPS_PULL);',
              "return 0;}"]
    src.write_text("\n".join(lines))
    exe = tmp_path / "layout"
    subprocess.run(["gcc", "-I", str(ROOT / "include"), "-o", str(exe), str(src)], check=True)
    out = subprocess.run([str(exe)], check=True, capture_output=True, text=True).stdout.split()
    assert int(out[0]) == C.sizeof(binding.Config)
    for f, o in zip(fields, out[1:1 + len(fields)]):
        assert int(o) == getattr(binding.Config, f).offset, f
    rest = [int(x) for x in out[1 + len(fields):]]
    assert rest[0] == C.sizeof(binding.Event) == 16
    assert rest[1] == binding.EVENT_LOG_DTYPE.itemsize
    assert rest[2] == binding.EVENT_LOG_DTYPE.fields["t"][1]
    assert rest[3] == binding.EVENT_LOG_DTYPE.fields["gps_lag"][1]
    assert rest[4] == binding.EVENT_LOG_DTYPE.fields["pushed"][1]
    lr = binding.LAUNCH_RECORD_DTYPE
    assert rest[5:10] == [lr.itemsize] + [lr.fields[f][1] for f in ("kind", "events", "bytes_per_param", "ms")]
    assert rest[10] == len(binding.KERNEL_NAMES) and rest[11] == binding.K_GPS_PULL
    from paper_2506_04531_b200.inputs import trace as tr
    assert tr.EVENT_DTYPE.itemsize == 16 and tr.EVENT_DTYPE.fields["time_ns"][1] == 8


def test_default_config_and_messages(lib):
    from paper_2506_04531_b200 import binding
    cfg = binding.Config()
    lib.halos_default_config(C.byref(cfg))
    assert cfg.struct_size == C.sizeof(binding.Config)
    assert (round(cfg.eta_l, 6), round(cfg.beta_l, 6), round(cfg.eta_g, 6), round(cfg.beta_g, 6),
            round(cfg.alpha, 6), cfg.K) == (0.2, 0.9, 0.15, 0.5, 0.25, 32)
    assert lib.halos_strerror(0) == b"ok"
    assert b"order" in lib.halos_strerror(binding.ERR_BAD_STATE)
    assert lib.halos_destroy(None) == binding.OK


def test_create_rejects_bad_arguments_without_touching_a_device(lib):
    from paper_2506_04531_b200 import binding
    out = C.c_void_p()
    assert lib.halos_create(None, None, C.byref(out)) == binding.ERR_INVALID_ARG
    cfg = binding.Config()
    lib.halos_default_config(C.byref(cfg))
    dummy = C.c_void_p(256)
    assert lib.halos_create(C.byref(cfg), dummy, C.byref(out)) == binding.ERR_INVALID_ARG   # empty config
    assert b"empty" in lib.halos_last_error(None)
    wl = (C.c_uint32 * 2)(0, 5)
    tn = (C.c_uint64 * 1)(16)
    cfg.n_lps, cfg.n_workers, cfg.n_tensors = 2, 2, 1
    cfg.worker_lps, cfg.tensor_numel = wl, tn
    assert lib.halos_create(C.byref(cfg), dummy, C.byref(out)) == binding.ERR_INVALID_ARG   # worker_lps[1] = 5
    wl[1] = 1
    cfg.struct_size = 8
    assert lib.halos_create(C.byref(cfg), dummy, C.byref(out)) == binding.ERR_INVALID_ARG   # ABI size mismatch
    cfg.struct_size = C.sizeof(binding.Config)
    cfg.chunk_elems = 6
    assert lib.halos_create(C.byref(cfg), dummy, C.byref(out)) == binding.ERR_INVALID_ARG
    cfg.chunk_elems = 0
    import torch
    if not torch.cuda.is_available():
        # valid arguments but no device: the library must refuse, there is no CPU path
        assert lib.halos_create(C.byref(cfg), dummy, C.byref(out)) == binding.ERR_CUDA
        assert b"no CPU path" in lib.halos_last_error(None)
        with pytest.raises(binding.HalosError):
            binding.Halos(torch.zeros(4), [0])


def test_product_never_imports_the_oracle():
    """The CUDA package must not reach the oracle in any way."""
    pkg = ROOT / "paper_2506_04531_b200"
    for path in list(pkg.rglob("*.py")) + list(pkg.rglob("*.cu")) + list(pkg.rglob("*.cuh")) + [ROOT / "include" / "halos.h"]:
        text = path.read_text()
        assert "import oracle" not in text and "from oracle" not in text and "halos_oracle" not in text, path
    code = ("import sys; sys.path.insert(0, %r); import paper_2506_04531_b200.binding, paper_2506_04531_b200.inputs; "
            "assert not any(m == 'oracle' or m.startswith('oracle.') for m in sys.modules)") % str(ROOT)
    subprocess.run([sys.executable, "-c", code], check=True)
