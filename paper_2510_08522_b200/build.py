"""In-tree build of the two shared objects (nvcc, sm_100a only):
    lib/libdmx.so      the gradient-step library (C ABI of include/dmx.h)
    lib/libdmx_gen.so  the synthetic-input fill kernels
Run as `python -m paper_2510_08522_b200.build [--force] [--verbose]`.
"""
from __future__ import annotations

import os
import subprocess
import sys

_PKG = os.path.dirname(os.path.abspath(__file__))
_ROOT = os.path.dirname(_PKG)
CSRC = os.path.join(_PKG, "csrc")
LIBDIR = os.path.join(_PKG, "lib")
INCLUDE = os.path.join(_ROOT, "include")

NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
              "-shared", "-Xcompiler", "-fPIC", "-I", INCLUDE, "-I", CSRC]

TARGETS = {
    "libdmx.so": (["dmx.cu", "dmx_static.cu", "dmx_agg.cu", "dmx_ctl.cu"], ["dmx_kernels.cuh", "dmx_host.h", os.path.join(INCLUDE, "dmx.h")]),
    "libdmx_gen.so": (["dmx_gen.cu"], []),
}


def _nvcc() -> str:
    for cand in (os.environ.get("NVCC"), "/usr/local/cuda/bin/nvcc", "nvcc"):
        if cand and (os.path.isabs(cand) and os.path.exists(cand) or not os.path.isabs(cand)):
            return cand
    return "nvcc"


def lib_path(name: str) -> str:
    return os.path.join(LIBDIR, name)


def build(force: bool = False, verbose: bool = False) -> None:
    os.makedirs(LIBDIR, exist_ok=True)
    for name, (srcs, deps) in TARGETS.items():
        out = lib_path(name)
        srcs_abs = [os.path.join(CSRC, s) for s in srcs]
        deps_abs = srcs_abs + [d if os.path.isabs(d) else os.path.join(CSRC, d) for d in deps]
        if not force and os.path.exists(out) and all(os.path.getmtime(out) >= os.path.getmtime(d) for d in deps_abs):
            continue
        cmd = [_nvcc()] + NVCC_FLAGS + (["-Xptxas", "-v"] if verbose else []) + srcs_abs + ["-o", out + ".tmp"]
        if verbose:
            print(" ".join(cmd), flush=True)
        subprocess.check_call(cmd)
        os.replace(out + ".tmp", out)


if __name__ == "__main__":
    build(force="--force" in sys.argv, verbose="--verbose" in sys.argv)
