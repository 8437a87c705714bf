"""Compile libsamdraft.so in-tree with nvcc for sm_100a (cross-compiles without a GPU)."""
from __future__ import annotations

import glob
import os
import subprocess

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
# SAMDRAFT_VARIANT=counters makes the package load a second build of the same sources with -DSAM_COUNTERS
# (operation counters in the step kernels, for tests and for the benchmark's latency bound).
VARIANT = os.environ.get("SAMDRAFT_VARIANT", "")
VARIANTS = {"": ("libsamdraft.so", []), "counters": ("libsamdraft_counters.so", ["-DSAM_COUNTERS"])}
LIB = os.path.join(HERE, VARIANTS[VARIANT][0])
SOURCES = ["static_builder.cpp", "static_store.cu", "batch.cu", "step.cu", "probes.cu", "noalloc.cu", "accept.cu", "tree.cu"]
NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
              "-Xcompiler", "-fPIC", "-shared", "--cudart", "shared"]


def _sources():
    return [os.path.join(CSRC, s) for s in SOURCES if os.path.exists(os.path.join(CSRC, s))]


def _stale(lib: str) -> bool:
    if not os.path.exists(lib):
        return True
    t = os.path.getmtime(lib)
    deps = _sources() + glob.glob(os.path.join(CSRC, "*.h")) + \
        [os.path.join(os.path.dirname(HERE), "include", "samdraft.h")]
    return any(os.path.getmtime(d) > t for d in deps)


def build(force: bool = False, verbose: bool = False, variant: str | None = None) -> str:
    """Build the library (the variant the package loads, unless another is named) if it is missing or
    older than its sources; returns its path."""
    name, defines = VARIANTS[VARIANT if variant is None else variant]
    lib = os.path.join(HERE, name)
    if force or _stale(lib):
        nvcc = os.environ.get("NVCC", "nvcc")
        tmp = lib + ".tmp%d" % os.getpid()
        cmd = [nvcc] + NVCC_FLAGS + defines + (["-Xptxas", "-v"] if verbose else []) + ["-o", tmp] + _sources()
        subprocess.check_call(cmd, cwd=CSRC)
        os.replace(tmp, lib)
    return lib


if __name__ == "__main__":
    for v in VARIANTS:
        print(build(force=True, verbose=True, variant=v))
