"""Build libsoftsync_ps.so (the C-ABI library with its sm_100a kernels) in-tree with nvcc."""
from __future__ import annotations

import os
import shutil
import subprocess

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libsoftsync_ps.so")
SOURCES = ["softsync_ps.cu"]
HEADERS = [os.path.join(CSRC, "update_kernels.cuh"),
           os.path.join(os.path.dirname(HERE), "include", "softsync_ps.h")]

NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
              "-shared", "-Xcompiler", "-fPIC", "-cudart", "static"]


def nvcc() -> str:
    exe = shutil.which("nvcc") or "/usr/local/cuda/bin/nvcc"
    if not os.path.exists(exe):
        raise RuntimeError("nvcc not found: the library cannot be built")
    return exe


def is_stale() -> bool:
    if not os.path.exists(LIB):
        return True
    deps = [os.path.join(CSRC, s) for s in SOURCES] + HEADERS
    return any(os.path.getmtime(d) > os.path.getmtime(LIB) for d in deps)


def build(force: bool = False, verbose: bool = False) -> str:
    if not force and not is_stale():
        return LIB
    cmd = [nvcc()] + NVCC_FLAGS + (["-Xptxas", "-v"] if verbose else []) + \
          ["-o", LIB] + [os.path.join(CSRC, s) for s in SOURCES]
    subprocess.run(cmd, check=True)
    return LIB


def ensure_built() -> str:
    """Build the library if it is missing or older than its sources.  A stale library is kept when the
    rebuild fails (no compiler on this machine); a missing one is an error."""
    if not os.path.exists(LIB):
        return build(force=True)
    if is_stale():
        try:
            return build(force=True)
        except Exception:
            return LIB
    return LIB


if __name__ == "__main__":
    import sys
    print(build(force=True, verbose="-v" in sys.argv))
