"""Compile the CPU oracle (plain C) into oracle/libsbc_oracle.so.

Test infrastructure only: the CUDA library neither links nor loads this.
Run as ``python oracle/build.py`` or call :func:`build`.
"""
import os
import subprocess

HERE = os.path.dirname(os.path.abspath(__file__))
SRC = os.path.join(HERE, "sbc_oracle.c")
LIB = os.path.join(HERE, "libsbc_oracle.so")


def build(force: bool = False) -> str:
    """Build the shared object if it is missing or older than its sources."""
    deps = [SRC, os.path.join(HERE, "sbc_oracle.h")]
    if not force and os.path.exists(LIB):
        if all(os.path.getmtime(LIB) >= os.path.getmtime(d) for d in deps):
            return LIB
    cmd = [
        "gcc", "-O2", "-std=c11", "-Wall", "-Wextra", "-fPIC", "-shared",
        # no fused multiply-add, no value-changing optimisation: every fp32
        # operation in the oracle is the single IEEE operation it is written as
        "-ffp-contract=off", "-fno-fast-math",
        "-o", LIB, SRC, "-lm",
    ]
    subprocess.run(cmd, check=True, cwd=HERE)
    return LIB


if __name__ == "__main__":
    print(build(force=True))
