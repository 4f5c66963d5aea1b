"""Builds libswapmoe.so (the C-ABI CUDA library) in-tree with nvcc for sm_100a."""
from __future__ import annotations

import os
import subprocess
import sys

_HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(_HERE, "csrc")
LIB = os.path.join(_HERE, "libswapmoe.so")
TRACE_LIB = os.path.join(_HERE, "libswapmoe_trace.so")
SOURCES = ["api.cu", "route_static.cu"]
NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
              "-Xcompiler", "-fPIC", "-shared", "-cudart", "static"]


def _newest_source_mtime() -> float:
    m = 0.0
    for root in (CSRC, os.path.join(os.path.dirname(_HERE), "include")):
        for fn in os.listdir(root):
            m = max(m, os.path.getmtime(os.path.join(root, fn)))
    return m


def build(force: bool = False, verbose: bool = False, trace: bool = False) -> str:
    """Compile if the library is missing or older than any source; returns its path.

    trace=True builds libswapmoe_trace.so instead: the same kernels with %globaltimer stamps at their
    phase boundaries (-DSWAPMOE_TRACE) and the extra export swapmoe_debug_trace; select it with
    SWAPMOE_LIB=<path> to draw a timeline of one forward.  Never the default: the stamps cost time."""
    LIB = TRACE_LIB if trace else globals()["LIB"]
    if not force and os.path.exists(LIB) and os.path.getmtime(LIB) >= _newest_source_mtime():
        return LIB
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    tmp = LIB + ".tmp.%d" % os.getpid()
    cmd = [nvcc] + NVCC_FLAGS + (["-Xptxas", "-v"] if verbose else []) + (["-DSWAPMOE_TRACE"] if trace else []) + \
          ["-o", tmp] + [os.path.join(CSRC, s) for s in SOURCES]
    r = subprocess.run(cmd, capture_output=True, text=True)
    if verbose or r.returncode != 0:
        sys.stderr.write(r.stdout + r.stderr)
    if r.returncode != 0:
        raise RuntimeError("nvcc failed building libswapmoe.so")
    os.replace(tmp, LIB)
    return LIB


if __name__ == "__main__":
    print(build(force=True, verbose="-v" in sys.argv, trace="--trace" in sys.argv))
