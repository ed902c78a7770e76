"""Builds libcfi.so (the C-ABI library of include/cfi.h) in-tree with nvcc for sm_100a."""
from __future__ import annotations

import os
import subprocess
import sys

_PKG = os.path.dirname(os.path.abspath(__file__))
_ROOT = os.path.dirname(_PKG)
CSRC = os.path.join(_PKG, "csrc")
INCLUDE = os.path.join(_ROOT, "include")
LIB = os.path.join(_PKG, "libcfi.so")
SOURCES = ["cfi_pack.cpp", "cfi_layer.cu", "cfi_probe.cu", "cfi_srigl_update.cu"]


def _newest_source_mtime() -> float:
    paths = [os.path.join(CSRC, f) for f in os.listdir(CSRC)] + [os.path.join(INCLUDE, "cfi.h")]
    return max(os.path.getmtime(p) for p in paths)


def nvcc_command(out: str, verbose_ptxas: bool = False):
    cmd = ["nvcc", "-gencode", "arch=compute_100a,code=sm_100a", "-O3", "-std=c++17", "-lineinfo",
           "-Xcompiler", "-fPIC", "-shared", "-I", INCLUDE, "-I", CSRC]
    if verbose_ptxas:
        cmd += ["-Xptxas", "-v"]
    cmd += ["-o", out] + [os.path.join(CSRC, s) for s in SOURCES] + ["-lcudart"]
    return cmd


def build(force: bool = False, verbose: bool = False) -> str:
    """Compile if the shared object is missing or older than any source; return its path."""
    if force or not os.path.exists(LIB) or os.path.getmtime(LIB) < _newest_source_mtime():
        tmp = LIB + f".tmp{os.getpid()}"
        r = subprocess.run(nvcc_command(tmp, verbose), capture_output=True, text=True)
        if verbose:
            sys.stderr.write(r.stderr)
        if r.returncode != 0:
            raise RuntimeError("nvcc failed:\n" + r.stdout + r.stderr)
        os.replace(tmp, LIB)
    return LIB


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv))
