"""Builds the C-ABI CUDA libraries in-tree with nvcc for sm_100a:
librkv.so (the RefreshKV attention path) and libllama_harness.so (the decoder kernels of the end-to-end workload)."""
from __future__ import annotations

import glob
import os
import subprocess
import sys

PKG = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(PKG)
LIB = os.path.join(PKG, "librkv.so")
HARNESS_LIB = os.path.join(PKG, "libllama_harness.so")
TARGETS = {LIB: "csrc", HARNESS_LIB: "csrc_harness"}


def sources(sub: str = "csrc") -> list:
    return sorted(glob.glob(os.path.join(PKG, sub, "*.cu")))


def needs_build(lib: str = LIB) -> bool:
    if not os.path.exists(lib):
        return True
    sub = TARGETS[lib]
    t = os.path.getmtime(lib)
    deps = (sources(sub) + glob.glob(os.path.join(PKG, sub, "*.h")) + glob.glob(os.path.join(PKG, sub, "*.cuh")) +
            glob.glob(os.path.join(ROOT, "include", "*.h")))
    return any(os.path.getmtime(d) > t for d in deps)


def _compile(lib: str, verbose: bool) -> None:
    sub = TARGETS[lib]
    nvcc = os.environ.get("NVCC", "nvcc")
    cmd = [nvcc, "-std=c++17", "-O3", "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo",
           "-Xcompiler", "-fPIC", "-shared", "-I", os.path.join(ROOT, "include"), "-I", os.path.join(PKG, sub),
           "-o", lib] + sources(sub)
    if verbose:
        cmd += ["-Xptxas", "-v"]
    r = subprocess.run(cmd, capture_output=True, text=True)
    if r.returncode != 0:
        raise RuntimeError("nvcc failed:\n" + r.stdout + r.stderr)
    if verbose:
        sys.stderr.write(r.stdout + r.stderr)


def build(force: bool = False, verbose: bool = False) -> str:
    """Compile every .cu under csrc/ and csrc_harness/ into their shared libraries; returns librkv's path."""
    for lib in TARGETS:
        if force or needs_build(lib):
            _compile(lib, verbose)
    return LIB


if __name__ == "__main__":
    print(build(force=True, verbose="-v" in sys.argv))
