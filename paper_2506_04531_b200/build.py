"""Builds the CUDA libraries of this package in-tree with nvcc for sm_100a.

    python -m paper_2506_04531_b200.build [--force] [--verbose]

libhalos_b200.so         the product: C ABI of include/halos.h (csrc/)
libhalos_inputs.so       CUDA twin of the synthetic input generator (inputs/csrc/), harness only
"""
from __future__ import annotations

import os
import subprocess
import sys
from pathlib import Path

PKG = Path(__file__).resolve().parent
ROOT = PKG.parent
INCLUDE = ROOT / "include"

NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
              "-shared", "-Xcompiler", "-fPIC", "-cudart", "static"]

TARGETS = {
    "halos": dict(out=PKG / "libhalos_b200.so", src=[PKG / "csrc" / "halos.cu", PKG / "csrc" / "halos_noalloc.cu"],
                  deps=[PKG / "csrc" / "halos_kernels.cuh", INCLUDE / "halos.h"]),
    "inputs": dict(out=PKG / "inputs" / "libhalos_inputs.so", src=[PKG / "inputs" / "csrc" / "synth_inputs.cu"],
                   deps=[]),
}


def _stale(t) -> bool:
    out = t["out"]
    if not out.exists():
        return True
    newest = max(p.stat().st_mtime for p in t["src"] + t["deps"])
    return out.stat().st_mtime < newest


def build(force: bool = False, verbose: bool = False, which=None) -> None:
    nvcc = os.environ.get("NVCC", "nvcc")
    for name, t in TARGETS.items():
        if which and name not in which:
            continue
        if not all(p.exists() for p in t["src"]):
            continue
        if not force and not _stale(t):
            continue
        tmp = t["out"].with_suffix(f".so.tmp{os.getpid()}")
        cmd = [nvcc, *NVCC_FLAGS, "-I", str(INCLUDE), "-o", str(tmp), *map(str, t["src"])]
        if verbose:
            cmd.insert(1, "-Xptxas")
            cmd.insert(2, "-v")
            print(" ".join(cmd), flush=True)
        subprocess.run(cmd, check=True)
        os.replace(tmp, t["out"])


if __name__ == "__main__":
    build(force="--force" in sys.argv, verbose="--verbose" in sys.argv)
