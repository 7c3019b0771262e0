"""Compile the C part of the oracle with gcc (test infrastructure; not part of the product)."""
from __future__ import annotations

import os
import subprocess

_HERE = os.path.dirname(os.path.abspath(__file__))
SOURCES = [os.path.join(_HERE, "regional_block.c"), os.path.join(_HERE, "dense_block.c")]
LIB = os.path.join(_HERE, "libfd_oracle.so")


def build(force: bool = False) -> str:
    """Build ``libfd_oracle.so`` next to the sources if it is missing or stale."""
    stale = force or not os.path.exists(LIB) or any(
        os.path.getmtime(s) > os.path.getmtime(LIB) for s in SOURCES)
    if stale:
        # -ffp-contract=off and no -march: no fused multiply-add is formed, so the regional and
        # the dense program round identically wherever they state the same arithmetic.
        cmd = ["gcc", "-O2", "-fopenmp", "-ffp-contract=off", "-fPIC", "-shared", "-std=c11",
               "-o", LIB + ".tmp"] + SOURCES + ["-lm"]
        subprocess.run(cmd, check=True)
        os.replace(LIB + ".tmp", LIB)
    return LIB


if __name__ == "__main__":
    print(build(force=True))
