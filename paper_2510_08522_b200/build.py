"""In-tree build of the shared objects (nvcc, sm_100a only):
    lib/libdmx.so          the gradient-step library (C ABI of include/dmx.h)
    lib/libdmx_gen.so      the synthetic-input fill kernels
    lib/libdmx_checked.so  (with --checked) the gradient-step library compiled with -DDMX_DEBUG:
                           every index into the tables and the scratch is range-tested on the
                           device; a violation sets DMX_FLAG_BOUNDS in the state vector, never a trap
Run as `python -m paper_2510_08522_b200.build [--force] [--verbose] [--checked]`.
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


CHECKED = {"libdmx_checked.so": TARGETS["libdmx.so"]}


def build(force: bool = False, verbose: bool = False, checked: bool = False) -> None:
    """Compile the targets that are missing or older than their sources; the nvcc runs of different
    targets go side by side (each takes about a minute and a half, nearly all of it in dmx.cu)."""
    from concurrent.futures import ThreadPoolExecutor
    os.makedirs(LIBDIR, exist_ok=True)
    targets = dict(TARGETS)
    if checked:
        targets.update(CHECKED)
    jobs = []
    for name, (srcs, deps) in targets.items():
        out = lib_path(name)
        srcs_abs = [os.path.join(CSRC, s) for s in srcs]
        deps_abs = srcs_abs + [d if os.path.isabs(d) else os.path.join(CSRC, d) for d in deps]
        if not force and os.path.exists(out) and all(os.path.getmtime(out) >= os.path.getmtime(d) for d in deps_abs):
            continue
        tmp = "%s.%d.tmp" % (out, os.getpid())
        cmd = ([_nvcc()] + NVCC_FLAGS + (["-DDMX_DEBUG"] if name in CHECKED else []) +
               (["-Xptxas", "-v"] if verbose else []) + srcs_abs + ["-o", tmp])
        jobs.append((cmd, tmp, out))

    def run(job):
        cmd, tmp, out = job
        if verbose:
            print(" ".join(cmd), flush=True)
        subprocess.check_call(cmd)
        os.replace(tmp, out)

    if jobs:
        with ThreadPoolExecutor(max_workers=1 if verbose else len(jobs)) as pool:   # verbose: keep ptxas' output in order
            for _ in pool.map(run, jobs):       # re-raises the first failure
                pass


if __name__ == "__main__":
    build(force="--force" in sys.argv, verbose="--verbose" in sys.argv, checked="--checked" in sys.argv)
