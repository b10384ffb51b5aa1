"""Compile the oracle's C part (plain gcc, no CUDA).  Test infrastructure only."""
from __future__ import annotations

import os
import subprocess

HERE = os.path.dirname(os.path.abspath(__file__))
SRCS = [os.path.join(HERE, "transformer.c"), os.path.join(HERE, "sampling.c")]
LIB = os.path.join(HERE, "liboracle.so")


def build(force: bool = False) -> str:
    """Build ``liboracle.so`` beside the source if it is missing or stale; return its path.

    ``-ffp-contract=off`` keeps every multiply and add a separately rounded
    fp32 operation, so the oracle's results do not depend on whether the
    host CPU has fused multiply-add.
    """
    if not force and os.path.exists(LIB) and os.path.getmtime(LIB) >= max(os.path.getmtime(s) for s in SRCS):
        return LIB
    cmd = ["gcc", "-O3", "-march=x86-64-v3", "-ffp-contract=off", "-fopenmp", "-fPIC", "-shared",
           "-Wall", "-o", LIB] + SRCS + ["-lm"]
    subprocess.run(cmd, check=True)
    return LIB


if __name__ == "__main__":
    print(build(force=True))
