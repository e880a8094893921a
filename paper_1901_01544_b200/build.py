"""Builds the C-ABI library libiwp.so in-tree with nvcc for sm_100a (cross-compiles without a GPU)."""
from __future__ import annotations

import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libiwp.so")
SOURCES = [os.path.join(CSRC, "iwp_api.cu")]
DEPS = SOURCES + [os.path.join(CSRC, f) for f in ("iwp_device.cuh", "iwp_stream.cuh", "iwp_sample.cuh", "iwp_select.cuh", "iwp_reduce.cuh",
                                            "iwp_threshold.cuh", "iwp_wire.cuh", "iwp_plan.hpp")] + [
    os.path.join(os.path.dirname(HERE), "include", "iwp.h")
]

NVCC_FLAGS = [
    "-gencode", "arch=compute_100a,code=sm_100a",
    "-lineinfo", "-O3", "-std=c++17",
    # IEEE arithmetic: no FMA contraction, correctly rounded division, denormals kept
    "-fmad=false", "-prec-div=true", "-prec-sqrt=true", "-ftz=false",
    "-Xcompiler", "-fPIC", "-shared",
]


# The same library with every computed index range-checked and the histogram counts checked for conservation
# (a failed check sets the status word; nothing traps).  Loaded instead of libiwp.so when IWP_LIB_VARIANT=debug.
LIB_DEBUG = os.path.join(HERE, "libiwp_debug.so")


def stale(lib: str = LIB) -> bool:
    if not os.path.exists(lib):
        return True
    t = os.path.getmtime(lib)
    return any(os.path.getmtime(d) > t for d in DEPS)


def build(force: bool = False, verbose: bool = False, debug: bool = False) -> str:
    lib = LIB_DEBUG if debug else LIB
    if not force and not stale(lib):
        return lib
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    cmd = ([nvcc] + NVCC_FLAGS + (["-DIWP_DEBUG_CHECKS"] if debug else []) + (["-Xptxas", "-v"] if verbose else []) +
           SOURCES + ["-o", lib + ".tmp"])
    r = subprocess.run(cmd, capture_output=True, text=True)
    if r.returncode != 0:
        sys.stderr.write(r.stdout + r.stderr)
        raise RuntimeError(f"nvcc failed building {os.path.basename(lib)}")
    if verbose:
        sys.stderr.write(r.stdout + r.stderr)
    os.replace(lib + ".tmp", lib)
    return lib


if __name__ == "__main__":
    print(build(force=True, verbose="-v" in sys.argv, debug="--debug" in sys.argv))
