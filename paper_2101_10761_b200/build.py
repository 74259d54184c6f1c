"""Build the C-ABI library in-tree with nvcc for sm_100a.

libsidco.so is the product.  Two more builds of the same sources exist for tests and profiling:
libsidco_profile.so (-DSIDCO_PROFILE: device timestamps at phase boundaries) and libsidco_check.so
(-DSIDCO_BOUNDS_CHECK: every index into a caller or workspace buffer is range-checked on the device).
"""
from __future__ import annotations

import glob
import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
SOURCES = sorted(glob.glob(os.path.join(CSRC, "*.cu")))
DEPS = SOURCES + sorted(glob.glob(os.path.join(CSRC, "*.cuh"))) + \
    sorted(glob.glob(os.path.join(os.path.dirname(HERE), "include", "*.h")))
VARIANTS = {"": [], "profile": ["-DSIDCO_PROFILE"], "check": ["-DSIDCO_BOUNDS_CHECK"]}


def lib_path(variant: str = "") -> str:
    return os.path.join(HERE, "libsidco%s.so" % ("_" + variant if variant else ""))


LIB = lib_path()


def nvcc_path() -> str:
    cand = os.path.join(os.environ.get("CUDA_HOME", "/usr/local/cuda"), "bin", "nvcc")
    return cand if os.path.exists(cand) else "nvcc"


def _command(variant: str, verbose: bool):
    cmd = [nvcc_path(), "-std=c++17", "-O3", "-lineinfo",
           "-gencode", "arch=compute_100a,code=sm_100a",
           "-Xcompiler", "-fPIC", "-shared", "-cudart", "shared"] + VARIANTS[variant] + \
          ["-o", lib_path(variant)] + SOURCES
    if verbose:
        cmd[1:1] = ["-Xptxas", "-v"]
    return cmd


def _stale(variant: str) -> bool:
    lib = lib_path(variant)
    return not os.path.exists(lib) or any(os.path.getmtime(lib) < os.path.getmtime(p) for p in DEPS)


def build(force: bool = False, verbose: bool = False, variants=("",)) -> str:
    """Compile the named variants (in parallel) if they are older than their sources."""
    jobs = [(v, subprocess.Popen(_command(v, verbose), stdout=subprocess.PIPE, stderr=subprocess.STDOUT, text=True))
            for v in variants if force or _stale(v)]
    for v, proc in jobs:
        out, _ = proc.communicate()
        if verbose:
            sys.stderr.write(out)
        if proc.returncode != 0:
            raise RuntimeError("nvcc failed for variant %r:\n%s" % (v, out))
    return lib_path(variants[0])


def build_all(force: bool = False) -> None:
    build(force=force, variants=tuple(VARIANTS))


if __name__ == "__main__":
    names = tuple(VARIANTS) if "--all" in sys.argv else ("",)
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv, variants=names))
