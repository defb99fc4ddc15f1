"""Build libsoftsync_ps.so (the C-ABI library with its sm_100a kernels) in-tree with nvcc."""
from __future__ import annotations

import hashlib
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


STAMP = LIB + ".hash"            # digest of the sources and flags the library was built from


def source_digest() -> str:
    h = hashlib.sha256(" ".join(NVCC_FLAGS).encode())
    for path in [os.path.join(CSRC, s) for s in SOURCES] + HEADERS:
        with open(path, "rb") as f:
            h.update(f.read())
    return h.hexdigest()


def is_stale() -> bool:
    """True unless the library exists and was built from exactly the present sources (file times are not
    trusted: a copied tree does not keep them)."""
    if not os.path.exists(LIB) or not os.path.exists(STAMP):
        return True
    with open(STAMP) as f:
        return f.read().strip() != source_digest()


def build(force: bool = False, verbose: bool = False) -> str:
    if not force and not is_stale():
        return LIB
    cmd = [nvcc()] + NVCC_FLAGS + (["-Xptxas", "-v"] if verbose else []) + \
          ["-o", LIB] + [os.path.join(CSRC, s) for s in SOURCES]
    if os.path.exists(STAMP):
        os.remove(STAMP)
    subprocess.run(cmd, check=True)
    with open(STAMP, "w") as f:
        f.write(source_digest() + "\n")
    return LIB


def ensure_built() -> str:
    """Build the library if it is missing or was built from other sources.  A failed rebuild raises: a
    library that does not match the header and the binding must not be loaded."""
    if is_stale():
        return build(force=True)
    return LIB


if __name__ == "__main__":
    import sys
    print(build(force=True, verbose="-v" in sys.argv))
