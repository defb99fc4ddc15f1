"""Compile the C reference into oracle/liboracle_softsync.so with gcc.

TEST INFRASTRUCTURE: building the checker is not using it.  -ffp-contract=off
keeps every fp32 multiply and add a separately rounded IEEE operation, which
is what the reference's definition of the update states.
"""
from __future__ import annotations

import os
import subprocess

HERE = os.path.dirname(os.path.abspath(__file__))
LIB = os.path.join(HERE, "liboracle_softsync.so")
SOURCES = ["softsync_oracle.c", "arrival_sim.c"]
DEPS = SOURCES + ["update_rule.inc"]


def build(force: bool = False) -> str:
    srcs = [os.path.join(HERE, s) for s in SOURCES]
    deps = [os.path.join(HERE, s) for s in DEPS]
    if not force and os.path.exists(LIB) and all(os.path.getmtime(LIB) >= os.path.getmtime(d) for d in deps):
        return LIB
    cmd = ["gcc", "-O2", "-std=c11", "-ffp-contract=off", "-fno-fast-math", "-fPIC", "-shared",
           "-Wall", "-Wextra", "-o", LIB] + srcs + ["-lm"]
    subprocess.run(cmd, check=True, cwd=HERE)
    return LIB


if __name__ == "__main__":
    print(build(force=True))
